// Update kernels of the SLIDE step (Algorithm 1 "Update weights with Adam"; Section 3.5: a
// momentum and a velocity array per weight and bias array; Section 2.1: gradients reach the
// active neurons only).
//
//   k_scan : turns the per-row "touched" bitmaps written by the forward kernel into ascending
//            lists of distinct rows (a prefix sum over popcounts), reduces the batch loss in a
//            fixed order and advances the Adam step count.
//   k_adam : one warp per distinct touched row.  The row's gradient is rebuilt on the fly from
//            the samples that touch it (a bit mask per row, walked in ascending sample order, so
//            the sum is deterministic and no floating-point atomics are used), then Adam is
//            applied to that row only.  Rows nobody touched are neither read nor written.
#include "common.cuh"

namespace dslide {

constexpr int SCAN_THREADS = 1024;
constexpr int ADAM_THREADS = 256;
constexpr int ADAM_WARPS = ADAM_THREADS / 32;
constexpr int MAX_HCHUNK = 8;

__global__ void __launch_bounds__(SCAN_THREADS)
k_scan(uint32_t* touched2, int nwords2, int32_t* uniq2, uint32_t* touched1, int nwords1, int32_t* uniq1,
       DevState* st, const float* loss, int B, float* loss_out, float beta1, float beta2, int dense, int N) {
  __shared__ int sh[SCAN_THREADS / 32 + 1];
  __shared__ float shf[SCAN_THREADS / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t* bm = blockIdx.x == 0 ? touched2 : touched1;
  const int nwords = blockIdx.x == 0 ? nwords2 : nwords1;
  int32_t* out = blockIdx.x == 0 ? uniq2 : uniq1;

  if (!(blockIdx.x == 0 && dense)) {
    const int chunk = (nwords + SCAN_THREADS - 1) / SCAN_THREADS;
    const int wbeg = tid * chunk, wend = min(nwords, wbeg + chunk);
    int cnt = 0;
    for (int w = wbeg; w < wend; ++w) cnt += __popc(bm[w]);
    int incl = cnt;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      int n = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += n;
    }
    if (lane == 31) sh[warp] = incl;
    __syncthreads();
    if (tid == 0) {
      int run = 0;
      for (int w = 0; w < SCAN_THREADS / 32; ++w) { int c = sh[w]; sh[w] = run; run += c; }
      sh[SCAN_THREADS / 32] = run;
    }
    __syncthreads();
    int pos = incl - cnt + sh[warp];
    for (int w = wbeg; w < wend; ++w) {
      uint32_t bits = bm[w];
      if (bits) bm[w] = 0u;                      // clean for the next step
      while (bits) {
        int b = __ffs(bits) - 1;
        out[pos++] = (w << 5) + b;
        bits &= bits - 1;
      }
    }
    if (tid == 0) {
      const int u = sh[SCAN_THREADS / 32];
      if (blockIdx.x == 0) { st->U2 = u; st->cum[2] += (unsigned long long)u; }
      else { st->U1 = u; st->cum[3] += (unsigned long long)u; }
    }
  } else if (tid == 0) {
    st->U2 = N;
    st->cum[2] += (unsigned long long)N;
  }

  if (blockIdx.x == 0) {
    // mean loss of the batch, summed in a fixed order
    float v = 0.f;
    for (int s = tid; s < B; s += SCAN_THREADS) v += loss[s];
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    if (lane == 0) shf[warp] = v;
    __syncthreads();
    if (tid == 0) {
      float r = 0.f;
      for (int w = 0; w < SCAN_THREADS / 32; ++w) r += shf[w];
      if (loss_out) *loss_out = r / (float)B;
      long long t = st->t + 1;
      st->t = t;
      st->bc1 = (float)(1.0 - pow((double)beta1, (double)t));
      st->bc2 = (float)(1.0 - pow((double)beta2, (double)t));
      st->last_sum_active = st->sum_active; st->sum_active = 0ull;
      st->last_nnz = st->nnz; st->nnz = 0ull;
      st->last_fetched = st->fetched; st->fetched = 0ull;
      st->cum[0] += 1ull; st->cum[1] += st->last_sum_active; st->cum[4] += st->last_nnz; st->cum[5] += st->last_fetched;
    }
  }
}

struct AdamParams {
  float *W1, *mW1, *vW1, *b1, *mb1, *vb1;
  float *W2, *mW2, *vW2, *b2, *mb2, *vb2;
  const float *h, *dh, *act_g;
  const int32_t *act_cnt, *act_ids;
  const int32_t *row_ptr, *col_idx;
  const float* vals;
  uint32_t *mask1, *mask2;
  const int32_t *uniq1, *uniq2;
  const DevState* st;
  int B, H, N, Wd, act_stride, dense;
  float lr, beta1, beta2, eps;
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

// acc += sum over the set bits b of `bits` (ascending) of coef[b] * src[(sbase + b) * H ...], where coef[b]
// lives in lane b.  Up to four rows are loaded before they are used, in order.
__device__ __forceinline__ void accumulate_word(float4 (&acc)[MAX_HCHUNK], float& csum, uint32_t bits, float coef,
                                                int sbase, const float* src, int H, int H4, int lane) {
  while (bits) {
    int b[4]; float g[4]; int n = 0;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      b[r] = -1; g[r] = 0.f;
      if (bits) { b[r] = __ffs(bits) - 1; bits &= bits - 1; n = r + 1; }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) g[r] = __shfl_sync(0xffffffffu, coef, b[r] < 0 ? 0 : b[r]);
#pragma unroll
    for (int q = 0; q < MAX_HCHUNK; ++q) {
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

__device__ __forceinline__ void adam_row(float* W, float* M, float* V, size_t row, const float4 (&acc)[MAX_HCHUNK],
                                         int H, int H4, int lane, const AdamParams& p, float bc1, float bc2) {
  float4* w4 = reinterpret_cast<float4*>(W + row * H);
  float4* m4 = reinterpret_cast<float4*>(M + row * H);
  float4* v4 = reinterpret_cast<float4*>(V + row * H);
#pragma unroll
  for (int q = 0; q < MAX_HCHUNK; ++q) {
    int c = lane + q * 32;
    if (c < H4) {
      float4 w = w4[c], m = m4[c], v = v4[c];
      adam1(w.x, m.x, v.x, acc[q].x, p.beta1, p.beta2, p.lr, p.eps, bc1, bc2);
      adam1(w.y, m.y, v.y, acc[q].y, p.beta1, p.beta2, p.lr, p.eps, bc1, bc2);
      adam1(w.z, m.z, v.z, acc[q].z, p.beta1, p.beta2, p.lr, p.eps, bc1, bc2);
      adam1(w.w, m.w, v.w, acc[q].w, p.beta1, p.beta2, p.lr, p.eps, bc1, bc2);
      w4[c] = w; m4[c] = m; v4[c] = v;
    }
  }
}

__global__ void __launch_bounds__(ADAM_THREADS) k_adam(const AdamParams p) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = p.H, H4 = H >> 2, B = p.B;
  const float bc1 = p.st->bc1, bc2 = p.st->bc2;

  if (blockIdx.x == 0) {
    // hidden bias: dense gradient, samples summed in ascending order
    for (int k = tid; k < H; k += ADAM_THREADS) {
      float g = 0.f;
      for (int s = 0; s < B; ++s) g += p.dh[(size_t)s * H + k];
      float w = p.b1[k], m = p.mb1[k], v = p.vb1[k];
      adam1(w, m, v, g, p.beta1, p.beta2, p.lr, p.eps, bc1, bc2);
      p.b1[k] = w; p.mb1[k] = m; p.vb1[k] = v;
    }
    return;
  }

  const int U2 = p.st->U2, U1 = p.st->U1;
  const int total = U2 + U1;
  const int nwB = (B + 31) >> 5;
  const int stride = (gridDim.x - 1) * ADAM_WARPS;
  for (int r = (blockIdx.x - 1) * ADAM_WARPS + warp; r < total; r += stride) {
    float4 acc[MAX_HCHUNK];
#pragma unroll
    for (int q = 0; q < MAX_HCHUNK; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
    float csum = 0.f;
    if (r < U2) {
      // ---- a row of W2 and its bias: dW2[j,:] = sum_s g[s,j] h[s,:], db2[j] = sum_s g[s,j] ----
      const int j = p.dense ? r : p.uniq2[r];
      if (p.dense) {
        for (int sb = 0; sb < B; sb += 32) {
          int s = sb + lane;
          float coef = s < B ? p.act_g[(size_t)s * p.act_stride + j] : 0.f;
          uint32_t bits = B - sb >= 32 ? 0xffffffffu : ((1u << (B - sb)) - 1u);
          accumulate_word(acc, csum, bits, coef, sb, p.h, H, H4, lane);
        }
      } else {
        uint32_t* mrow = p.mask2 + (size_t)j * p.Wd;
        for (int wb = 0; wb < nwB; wb += 32) {
          int wi = wb + lane;
          uint32_t word = wi < nwB ? mrow[wi] : 0u;
          if (word) mrow[wi] = 0u;                 // clean for the next step
          unsigned nz = __ballot_sync(0xffffffffu, word != 0u);
          while (nz) {
            int src = __ffs(nz) - 1;
            nz &= nz - 1;
            uint32_t bits = __shfl_sync(0xffffffffu, word, src);
            int sbase = (wb + src) << 5;
            float coef = 0.f;
            if ((bits >> lane) & 1u) {
              // lane b looks up the error of neuron j in sample sbase + b (ascending ids: binary search)
              int s = sbase + lane;
              const int32_t* ids = p.act_ids + (size_t)s * p.act_stride;
              int lo = 0, hi = p.act_cnt[s];
              while (lo < hi) { int mid = (lo + hi) >> 1; if (__ldg(ids + mid) < j) lo = mid + 1; else hi = mid; }
              if (lo < p.act_cnt[s] && __ldg(ids + lo) == j) coef = p.act_g[(size_t)s * p.act_stride + lo];
            }
            accumulate_word(acc, csum, bits, coef, sbase, p.h, H, H4, lane);
          }
        }
      }
      adam_row(p.W2, p.mW2, p.vW2, (size_t)j, acc, H, H4, lane, p, bc1, bc2);
      if (lane == 0) {
        float w = p.b2[j], m = p.mb2[j], v = p.vb2[j];
        adam1(w, m, v, csum, p.beta1, p.beta2, p.lr, p.eps, bc1, bc2);
        p.b2[j] = w; p.mb2[j] = m; p.vb2[j] = v;
      }
    } else {
      // ---- a row of W1: dW1[f,:] = sum_s x[s,f] dh[s,:] ----
      const int f = p.uniq1[r - U2];
      uint32_t* mrow = p.mask1 + (size_t)f * p.Wd;
      for (int wb = 0; wb < nwB; wb += 32) {
        int wi = wb + lane;
        uint32_t word = wi < nwB ? mrow[wi] : 0u;
        if (word) mrow[wi] = 0u;
        unsigned nz = __ballot_sync(0xffffffffu, word != 0u);
        while (nz) {
          int src = __ffs(nz) - 1;
          nz &= nz - 1;
          uint32_t bits = __shfl_sync(0xffffffffu, word, src);
          int sbase = (wb + src) << 5;
          float coef = 0.f;
          if ((bits >> lane) & 1u) {
            int s = sbase + lane;
            int lo = __ldg(p.row_ptr + s), end = __ldg(p.row_ptr + s + 1), hi = end;
            while (lo < hi) { int mid = (lo + hi) >> 1; if (__ldg(p.col_idx + mid) < f) lo = mid + 1; else hi = mid; }
            if (lo < end && __ldg(p.col_idx + lo) == f) coef = __ldg(p.vals + lo);
          }
          accumulate_word(acc, csum, bits, coef, sbase, p.dh, H, H4, lane);
        }
      }
      adam_row(p.W1, p.mW1, p.vW1, (size_t)f, acc, H, H4, lane, p, bc1, bc2);
    }
  }
}

cudaError_t launch_update(Ctx* c, int batch, const int32_t* row_ptr, const int32_t* col_idx, const float* vals,
                          float* loss_out) {
  {
    LaunchScope ls(c, KID_SCAN);
    k_scan<<<2, SCAN_THREADS, 0, c->stream>>>(c->touched2, (c->N + 31) / 32, c->uniq2, c->touched1, (c->D + 31) / 32,
                                              c->uniq1, c->dstate, c->loss, batch, loss_out, c->cfg.beta1,
                                              c->cfg.beta2, c->dense, c->N);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  AdamParams p;
  p.W1 = c->W1; p.mW1 = c->mW1; p.vW1 = c->vW1; p.b1 = c->b1; p.mb1 = c->mb1; p.vb1 = c->vb1;
  p.W2 = c->W2; p.mW2 = c->mW2; p.vW2 = c->vW2; p.b2 = c->b2; p.mb2 = c->mb2; p.vb2 = c->vb2;
  p.h = c->h; p.dh = c->dh; p.act_g = c->act_g; p.act_cnt = c->act_cnt; p.act_ids = c->act_ids;
  p.row_ptr = row_ptr; p.col_idx = col_idx; p.vals = vals;
  p.mask1 = c->mask1; p.mask2 = c->mask2; p.uniq1 = c->uniq1; p.uniq2 = c->uniq2; p.st = c->dstate;
  p.B = batch; p.H = c->H; p.N = c->N; p.Wd = c->Wd; p.act_stride = c->act_stride; p.dense = c->dense;
  p.lr = c->cfg.lr; p.beta1 = c->cfg.beta1; p.beta2 = c->cfg.beta2; p.eps = c->cfg.eps;
  {
    LaunchScope ls(c, KID_ADAM);
    k_adam<<<1 + c->num_sms * 4, ADAM_THREADS, 0, c->stream>>>(p);
  }
  return cudaGetLastError();
}

}  // namespace dslide
