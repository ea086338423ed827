// Initialisation and table (re)build (Algorithm 1: "Initialize layers with randomly generated
// weights", "Hash weights to hash tables", "Rebuild hash tables and hash functions"; Section 2.1
// phase 1; Section 3.1 "locally updated with a frequency schedule").
//
//   k_init_gauss   : weights ~ N(0, std^2) from the counter-based generator (Box-Muller).
//   k_draw_simhash / k_draw_dwta : the hash functions of rebuild count r.
//   k_hash_neurons : the L bucket codes of every row of W2 (same functions as the queries) and
//                    the size of every bucket.
//   k_bucket_scan  : bucket sizes -> bucket offsets (one block per table).
//   k_sort_hist / k_sort_scan / k_sort_scatter : a stable least-significant-digit radix sort of the
//                    neuron ids of each table by bucket code, so that every bucket lists its
//                    neurons in ascending id (the first `cap` of them are what a query reads).
#include "common.cuh"

namespace dslide {

// ------------------------------------------------------------------ weights
__global__ void k_init_gauss(float* w, long long n, uint64_t seed, uint64_t stream_id, double std) {
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long step = (long long)gridDim.x * blockDim.x;
  for (; i < n; i += step) {
    uint64_t a = ctr_rng(seed, stream_id, 0, 2ull * (uint64_t)i);
    uint64_t b = ctr_rng(seed, stream_id, 0, 2ull * (uint64_t)i + 1ull);
    double u1 = ((double)(a >> 11) + 0.5) * (1.0 / 9007199254740992.0);
    double u2 = ((double)(b >> 11) + 0.5) * (1.0 / 9007199254740992.0);
    w[i] = (float)(std * sqrt(-2.0 * log(u1)) * cos(6.283185307179586476925 * u2));
  }
}

cudaError_t launch_init_gauss(Ctx* c, float* w, int64_t n, uint64_t stream_id) {
  if (n <= 0) return cudaSuccess;
  {
    LaunchScope ls(c, KID_INIT);
    k_init_gauss<<<c->num_sms * 8, 256, 0, c->stream>>>(w, n, c->cfg.seed, stream_id, (double)c->cfg.init_std);
  }
  return cudaGetLastError();
}

// ------------------------------------------------------------------ hash functions
// SimHash: projection f has fn_len distinct coordinates (partial Fisher-Yates over 0..H-1, then
// sorted ascending) and a sign per coordinate.  One thread per projection; H <= 1024.
__global__ void k_draw_simhash(int32_t* idx, int32_t* sign, int KL, int H, int m, uint64_t seed, uint64_t r) {
  int f = blockIdx.x * blockDim.x + threadIdx.x;
  if (f >= KL) return;
  short perm[1024];
  for (int i = 0; i < H; ++i) perm[i] = (short)i;
  for (int i = 0; i < m; ++i) {
    uint64_t u = ctr_rng(seed, RNG_HASH, r, (uint64_t)f * 2ull * (uint64_t)m + (uint64_t)i);
    int j = i + (int)(u % (uint64_t)(H - i));
    short tmp = perm[i]; perm[i] = perm[j]; perm[j] = tmp;
  }
  for (int i = 1; i < m; ++i) {      // insertion sort of the chosen coordinates
    short v = perm[i];
    int q = i;
    while (q > 0 && perm[q - 1] > v) { perm[q] = perm[q - 1]; --q; }
    perm[q] = v;
  }
  for (int i = 0; i < m; ++i) {
    uint64_t u = ctr_rng(seed, RNG_HASH, r, (uint64_t)f * 2ull * (uint64_t)m + (uint64_t)m + (uint64_t)i);
    idx[(size_t)f * m + i] = perm[i];
    sign[(size_t)f * m + i] = (u & 1ull) ? 1 : -1;
  }
}

// DWTA: ceil(K*L*bin / H) random permutations of the coordinates, concatenated; hash function f
// reads entries [f*bin, (f+1)*bin).  One block per permutation: the swap partner of every position is drawn by
// its own thread (the generator is counter-based), then one thread applies the swaps from the last position down.
constexpr int DRAW_THREADS = 128;
__global__ void __launch_bounds__(DRAW_THREADS) k_draw_dwta(int32_t* idx, long long total, int H, uint64_t seed, uint64_t r) {
  extern __shared__ int draw_sm[];          // [H] permutation, [H] swap partners
  int* perm = draw_sm;
  int* partner = draw_sm + H;
  const int q = blockIdx.x;
  for (int i = threadIdx.x; i < H; i += DRAW_THREADS) {
    perm[i] = i;
    const uint64_t u = ctr_rng(seed, RNG_HASH, r, (uint64_t)q * (uint64_t)H + (uint64_t)i);
    partner[i] = i >= 1 ? (int)(u % (uint64_t)(i + 1)) : 0;
  }
  __syncthreads();
  if (threadIdx.x == 0)
    for (int i = H - 1; i >= 1; --i) {
      const int j = partner[i];
      const int tmp = perm[i]; perm[i] = perm[j]; perm[j] = tmp;
    }
  __syncthreads();
  for (int i = threadIdx.x; i < H; i += DRAW_THREADS) {
    const long long e = (long long)q * H + i;
    if (e < total) idx[e] = perm[i];
  }
}

cudaError_t launch_draw_hash(Ctx* c, int64_t r) {
  LaunchScope ls(c, KID_DRAW_HASH);
  if (c->cfg.hash_family == DSLIDE_SIMHASH) {
    k_draw_simhash<<<(c->KL + 63) / 64, 64, 0, c->stream>>>(c->hash_idx, c->hash_sign, c->KL, c->H, c->fn_len,
                                                           c->cfg.seed, (uint64_t)r);
  } else {
    long long total = (long long)c->KL * c->fn_len;
    int nperm = (int)((total + c->H - 1) / c->H);
    k_draw_dwta<<<nperm, DRAW_THREADS, 2 * c->H * sizeof(int), c->stream>>>(c->hash_idx, total, c->H, c->cfg.seed, (uint64_t)r);
  }
  return cudaGetLastError();
}

// ------------------------------------------------------------------ LSH-sampled hidden layer
// Projections over the D input coordinates (Section 3.6: the hidden layer as a sparse layer; Algorithm 1 retrieves
// active neurons for every layer): entry (c, p) is +1, -1 or 0 with probability 1/6, 1/6, 2/3, drawn by itself from
// the counter-based generator.
__global__ void k_draw_proj1(int8_t* proj, long long n, uint64_t seed, uint64_t r) {
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long step = (long long)gridDim.x * blockDim.x;
  for (; i < n; i += step) {
    const uint64_t u = ctr_rng(seed, RNG_HASH1, r, (uint64_t)i) % 6ull;
    proj[i] = u == 0 ? 1 : (u == 1 ? -1 : 0);
  }
}

cudaError_t launch_draw_proj1(Ctx* c, int64_t r) {
  if (c->L1 <= 0) return cudaSuccess;
  LaunchScope ls(c, KID_DRAW_HASH);
  k_draw_proj1<<<c->num_sms * 8, 256, 0, c->stream>>>(c->proj1, (long long)c->D * c->KL1, c->cfg.seed, (uint64_t)r);
  return cudaGetLastError();
}

// Codes of the hidden neurons: neuron k's weight vector is column k of W1.  A block owns 32 neurons (the lanes) and
// 16 projections (four per warp) and walks the input coordinates in ascending order, because the sums are sequential
// like the oracle's.  Tiles of H1_CT coordinates pass through shared memory: the 128-byte pieces of the rows of W1
// by cp.async, two tiles deep; the projections' entries as floats (+1, -1, 0), so that one fused multiply-add per
// (coordinate, projection) adds +w, -w or nothing -- fma(+-1, w, s) rounds like s +- w, and fma(0, w, s) is s.
constexpr int H1_THREADS = 128;
constexpr int H1_CT = 128;        // coordinates per tile
constexpr int H1_PB = 16;         // projections per block
__global__ void __launch_bounds__(H1_THREADS)
k_hash_hidden(const float* __restrict__ W1, const int8_t* __restrict__ proj, unsigned char* bits, int D, int H, int KL1) {
  __shared__ __align__(16) float tw[2][H1_CT][32];
  __shared__ __align__(16) float tf[2][H1_CT][H1_PB];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int k0 = blockIdx.x * 32, p0 = blockIdx.y * H1_PB;
  const int ntiles = (D + H1_CT - 1) / H1_CT;
  auto load_w = [&](int stage, int t) {        // 128 rows x 8 pieces of 16 bytes
    const int c0 = t * H1_CT;
    for (int e = tid; e < H1_CT * 8; e += H1_THREADS) {
      const int row = e >> 3, piece = e & 7;
      if (c0 + row < D && k0 + 4 * piece < H)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(&tw[stage][row][4 * piece])),
                     "l"(W1 + (size_t)(c0 + row) * H + k0 + 4 * piece) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  // the projections' entries of a tile: thread = coordinate, 16 bytes each, held in registers until the tile's turn
  signed char pe[H1_PB];
  auto load_p = [&](int t) {
    const int c = t * H1_CT + tid;
#pragma unroll
    for (int q = 0; q < H1_PB; ++q) pe[q] = (c < D && p0 + q < KL1) ? (signed char)__ldg(proj + (size_t)c * KL1 + p0 + q) : (signed char)0;
  };
  float s[4] = {0.f, 0.f, 0.f, 0.f};
  load_w(0, 0);
  load_p(0);
  for (int t = 0; t < ntiles; ++t) {
    const int st = t & 1;
#pragma unroll
    for (int q = 0; q < H1_PB; ++q) tf[st][tid][q] = (float)pe[q];
    if (t + 1 < ntiles) {
      load_w(st ^ 1, t + 1);
      load_p(t + 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    const int nc = min(H1_CT, D - t * H1_CT);
#pragma unroll 8
    for (int c = 0; c < nc; ++c) {
      const float w = tw[st][c][lane];
      const float4 e = *reinterpret_cast<const float4*>(&tf[st][c][4 * warp]);
      s[0] = __fmaf_rn(e.x, w, s[0]);
      s[1] = __fmaf_rn(e.y, w, s[1]);
      s[2] = __fmaf_rn(e.z, w, s[2]);
      s[3] = __fmaf_rn(e.w, w, s[3]);
    }
    __syncthreads();
  }
  const int k = k0 + lane;
  if (k < H)
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int p = p0 + 4 * warp + q;
      if (p < KL1) bits[(size_t)p * H + k] = s[q] >= 0.f ? 1 : 0;
    }
}

// One block per table: codes from the bits, bucket sizes, offsets, and every neuron to its bucket's start plus the
// number of lower-numbered neurons with the same code (ascending ids inside a bucket).  H <= 1024.
__global__ void __launch_bounds__(1024)
k_tables1(const unsigned char* bits, uint32_t* codes, int32_t* off, int32_t* ids, int H, int K1) {
  extern __shared__ int t1_smem[];          // [H] codes, [2^K1 + 1] offsets
  int* scode = t1_smem;
  int* soff = t1_smem + H;
  const int t = blockIdx.x, nb = 1 << K1, tid = threadIdx.x;
  for (int b = tid; b <= nb; b += blockDim.x) soff[b] = 0;
  __syncthreads();
  for (int k = tid; k < H; k += blockDim.x) {
    int code = 0;
    for (int q = 0; q < K1; ++q) code |= (int)bits[(size_t)(t * K1 + q) * H + k] << q;
    scode[k] = code;
    codes[(size_t)t * H + k] = (uint32_t)code;
    atomicAdd(&soff[code + 1], 1);
  }
  __syncthreads();
  if (tid == 0) {
    int run = 0;
    for (int b = 0; b <= nb; ++b) { run += soff[b]; soff[b] = run; }
  }
  __syncthreads();
  int32_t* o = off + (size_t)t * (nb + 1);
  for (int b = tid; b <= nb; b += blockDim.x) o[b] = soff[b];
  for (int k = tid; k < H; k += blockDim.x) {
    const int code = scode[k];
    int before = 0;
    for (int j = 0; j < k; ++j) before += scode[j] == code ? 1 : 0;
    ids[(size_t)t * H + soff[code] + before] = k;
  }
}

cudaError_t launch_build_tables1(Ctx* c) {
  if (c->L1 <= 0) return cudaSuccess;
  unsigned char* bits = reinterpret_cast<unsigned char*>(c->codes1n + (size_t)c->L1 * c->H);     // [KL1][H] after the codes
  {
    LaunchScope ls(c, KID_HASH_NEURONS);
    dim3 grid((c->H + 31) / 32, (c->KL1 + H1_PB - 1) / H1_PB);
    k_hash_hidden<<<grid, H1_THREADS, 0, c->stream>>>(c->W1, c->proj1, bits, c->D, c->H, c->KL1);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int smem = (c->H + (1 << c->K1) + 1) * (int)sizeof(int);
  if (smem > 48 * 1024) {
    e = cudaFuncSetAttribute(k_tables1, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
  }
  LaunchScope ls(c, KID_BUCKET_SCAN);
  k_tables1<<<c->L1, 1024, smem, c->stream>>>(bits, c->codes1n, c->bucket1_off, c->bucket1_ids, c->H, c->K1);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ codes of all neurons
constexpr int HN_ROWS = 32;
constexpr int HN_THREADS = 256;
constexpr int HN_WARPS = HN_THREADS / 32;
constexpr int HN_FN_SMEM_MAX = 96 * 1024;    // hash-function tables larger than this stay in global memory
constexpr size_t COUNT_SPLIT_BYTES = (size_t)64 << 20;   // bucket counters beyond this are counted table by table

// A block stages HN_ROWS rows of W2 in shared memory (padded, so that 32 threads reading the same
// column of 32 different rows hit 32 banks) and evaluates the L codes of each row: lane = row, the
// warps share out the tables.  The hash functions sit in shared memory too, 16 bits per coordinate
// (the top bit carries a negative SimHash sign), read as warp-wide broadcasts.
// keys[t][j] = code of neuron j in table t; counts[t][code + 1] += 1; with `ranks`, ranks[t][j] = the count before
// (the neuron's place inside its bucket, in order of arrival).
template <bool FN_SMEM>
__global__ void __launch_bounds__(HN_THREADS)
k_hash_neurons(const float* __restrict__ W2, const int32_t* __restrict__ hidx, const int32_t* __restrict__ hsign,
               uint32_t* keys, uint32_t* ranks, int32_t* counts, int N, int H, int K, int L, int family, int lg_bin,
               int fn_len, long long nb) {      // counts == nullptr: codes only (k_count_ranks counts afterwards)
  extern __shared__ __align__(16) unsigned char hn_smem[];
  float* tile = reinterpret_cast<float*>(hn_smem);                    // [HN_ROWS][H + 1]
  const int ld = H + 1;
  unsigned short* fn = reinterpret_cast<unsigned short*>(hn_smem + (((size_t)HN_ROWS * ld * 4 + 15) & ~(size_t)15));
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nfn = K * L * fn_len;
  if (FN_SMEM) {
    for (int e = threadIdx.x; e < nfn; e += HN_THREADS) {
      unsigned v = (unsigned)hidx[e];
      if (family == DSLIDE_SIMHASH && hsign[e] < 0) v |= 0x8000u;
      fn[e] = (unsigned short)v;
    }
  }
  const int ntiles = (N + HN_ROWS - 1) / HN_ROWS;
  for (int tl = blockIdx.x; tl < ntiles; tl += gridDim.x) {
    const int j0 = tl * HN_ROWS;
    const int rows = min(HN_ROWS, N - j0);
    __syncthreads();
    {
      const int H4 = H >> 2, total4 = rows * H4;
      const float4* src = reinterpret_cast<const float4*>(W2 + (size_t)j0 * H);
      for (int e = threadIdx.x; e < total4; e += HN_THREADS) {
        const float4 x = __ldg(src + e);
        const int r = e / H4, k = (e - r * H4) << 2;
        float* d = tile + r * ld + k;
        d[0] = x.x; d[1] = x.y; d[2] = x.z; d[3] = x.w;
      }
    }
    __syncthreads();
    if (lane < rows) {
      const float* v = tile + lane * ld;
      for (int t = warp; t < L; t += HN_WARPS) {
        uint32_t code = 0;
#pragma unroll 2
        for (int k = 0; k < K; ++k) {
          const int f = t * K + k;
          if (family == DSLIDE_SIMHASH) {
            float sum = 0.f;
            if (FN_SMEM) {
              const unsigned short* ix = fn + (size_t)f * fn_len;
              for (int i = 0; i < fn_len; ++i) {
                const unsigned e = ix[i];
                const float x = v[e & 0x7fffu];
                sum = __fadd_rn(sum, (e & 0x8000u) ? -x : x);
              }
            } else {
              const int32_t* ix = hidx + (size_t)f * fn_len;
              const int32_t* sg = hsign + (size_t)f * fn_len;
              for (int i = 0; i < fn_len; ++i) {
                const float x = v[__ldg(ix + i)];
                sum = __fadd_rn(sum, __ldg(sg + i) > 0 ? x : -x);
              }
            }
            code |= (sum >= 0.f ? 1u : 0u) << k;
          } else {
            int best = 0;
            float bv;
            if (FN_SMEM && fn_len == 8) {
              // bin of eight: the eight coordinates come in one 16-byte broadcast load
              const uint4 q = *reinterpret_cast<const uint4*>(fn + (size_t)f * 8);
              const float x0 = v[q.x & 0xffffu], x1 = v[q.x >> 16], x2 = v[q.y & 0xffffu], x3 = v[q.y >> 16];
              const float x4 = v[q.z & 0xffffu], x5 = v[q.z >> 16], x6 = v[q.w & 0xffffu], x7 = v[q.w >> 16];
              bv = x0;
              if (x1 > bv) { bv = x1; best = 1; }
              if (x2 > bv) { bv = x2; best = 2; }
              if (x3 > bv) { bv = x3; best = 3; }
              if (x4 > bv) { bv = x4; best = 4; }
              if (x5 > bv) { bv = x5; best = 5; }
              if (x6 > bv) { bv = x6; best = 6; }
              if (x7 > bv) { bv = x7; best = 7; }
            } else if (FN_SMEM) {
              const unsigned short* ix = fn + (size_t)f * fn_len;
              bv = v[ix[0]];
              for (int i = 1; i < fn_len; ++i) {
                const float x = v[ix[i]];
                if (x > bv) { bv = x; best = i; }
              }
            } else {
              const int32_t* ix = hidx + (size_t)f * fn_len;
              bv = v[__ldg(ix)];
              for (int i = 1; i < fn_len; ++i) {
                const float x = v[__ldg(ix + i)];
                if (x > bv) { bv = x; best = i; }
              }
            }
            code |= (uint32_t)best << (k * lg_bin);
          }
        }
        keys[(size_t)t * N + j0 + lane] = code;
        if (counts) {
          int32_t* cnt = counts + (size_t)t * (size_t)(nb + 1) + code + 1;
          if (ranks) ranks[(size_t)t * N + j0 + lane] = (uint32_t)atomicAdd(cnt, 1);
          else atomicAdd(cnt, 1);
        }
      }
    }
  }
}

// DWTA with bins of eight, hash functions in shared memory: the same tiles, but two rows per lane.  A tile holds
// 64 rows as 32 pairs (row r and row r + 32 interleaved per coordinate), so that one 8-byte load fetches a
// coordinate of both rows and the index arithmetic is shared; the two rows' winners are found side by side.
constexpr int HN2_ROWS = 64;

__device__ __forceinline__ void wta_step(float x, int i, float& bv, int& best) {
  if (x > bv) { bv = x; best = i; }          // strict: the lowest position wins ties
}

template <bool COUNT>      // COUNT = false: codes only, the counting is a pass of its own
__global__ void __launch_bounds__(HN_THREADS)
k_hash_neurons_dwta8(const float* __restrict__ W2, const int32_t* __restrict__ hidx, uint32_t* keys, uint32_t* ranks,
                     int32_t* counts, int N, int H, int K, int L, int lg_bin, long long nb) {
  extern __shared__ __align__(16) unsigned char hn_smem[];
  float2* tile = reinterpret_cast<float2*>(hn_smem);                  // [32 pairs][H + 1]
  const int ld = H + 1;
  unsigned short* fn = reinterpret_cast<unsigned short*>(hn_smem + (((size_t)32 * ld * 8 + 15) & ~(size_t)15));
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int nfn = K * L * 8;
  // Inside a tile coordinate k sits at place (k / 4) + (H / 4) * (k % 4): the four components of a 16-byte global
  // load then go to four distant places and a warp's stores spread over the banks.  The function table holds places.
  const int Hq = H >> 2;
  for (int e = threadIdx.x; e < nfn; e += HN_THREADS) {
    const int k = hidx[e];
    fn[e] = (unsigned short)((k >> 2) + Hq * (k & 3));
  }
  const int ntiles = (N + HN2_ROWS - 1) / HN2_ROWS;
  for (int tl = blockIdx.x; tl < ntiles; tl += gridDim.x) {
    const int j0 = tl * HN2_ROWS;
    const int rows = min(HN2_ROWS, N - j0);
    __syncthreads();
    {
      const int H4 = H >> 2, total4 = rows * H4;
      const float4* src = reinterpret_cast<const float4*>(W2 + (size_t)j0 * H);
      float* tile1 = reinterpret_cast<float*>(tile);
      for (int e = threadIdx.x; e < total4; e += HN_THREADS) {
        const float4 x = __ldg(src + e);
        const int r = e / H4, c4 = e - r * H4;
        float* d = tile1 + ((size_t)(r & 31) * ld + c4) * 2 + (r >> 5);
        d[0] = x.x; d[2 * H4] = x.y; d[4 * H4] = x.z; d[6 * H4] = x.w;
      }
    }
    __syncthreads();
    const bool live0 = lane < rows, live1 = lane + 32 < rows;
    if (live0) {
      const float2* v = tile + (size_t)lane * ld;
      uint32_t pr0 = 0, pr1 = 0;
      size_t pidx = 0;
      bool pend = false, pend1 = false;
      for (int t = warp; t < L; t += HN_WARPS) {
        uint32_t code0 = 0, code1 = 0;
        for (int k = 0; k < K; ++k) {
          const uint4 q = *reinterpret_cast<const uint4*>(fn + (size_t)(t * K + k) * 8);
          const float2 x0 = v[q.x & 0xffffu], x1 = v[q.x >> 16], x2 = v[q.y & 0xffffu], x3 = v[q.y >> 16];
          const float2 x4 = v[q.z & 0xffffu], x5 = v[q.z >> 16], x6 = v[q.w & 0xffffu], x7 = v[q.w >> 16];
          float a = x0.x, b = x0.y;
          int ia = 0, ib = 0;
          wta_step(x1.x, 1, a, ia); wta_step(x1.y, 1, b, ib);
          wta_step(x2.x, 2, a, ia); wta_step(x2.y, 2, b, ib);
          wta_step(x3.x, 3, a, ia); wta_step(x3.y, 3, b, ib);
          wta_step(x4.x, 4, a, ia); wta_step(x4.y, 4, b, ib);
          wta_step(x5.x, 5, a, ia); wta_step(x5.y, 5, b, ib);
          wta_step(x6.x, 6, a, ia); wta_step(x6.y, 6, b, ib);
          wta_step(x7.x, 7, a, ia); wta_step(x7.y, 7, b, ib);
          code0 |= (uint32_t)ia << (k * lg_bin);
          code1 |= (uint32_t)ib << (k * lg_bin);
        }
        // the ranks asked for in the previous round have arrived by now: they are stored a round late so that
        // no warp waits on its atomics
        if (pend) {
          ranks[pidx] = pr0;
          if (pend1) ranks[pidx + 32] = pr1;
        }
        keys[(size_t)t * N + j0 + lane] = code0;
        if (!COUNT) {                        // codes only: k_count_ranks counts afterwards, table by table
          if (live1) keys[(size_t)t * N + j0 + 32 + lane] = code1;
          continue;
        }
        int32_t* cnt = counts + (size_t)t * (size_t)(nb + 1) + 1;
        if (ranks) {
          pr0 = (uint32_t)atomicAdd(cnt + code0, 1);
          pidx = (size_t)t * N + j0 + lane;
          pend = true;
          pend1 = live1;
        } else {
          atomicAdd(cnt + code0, 1);
        }
        if (live1) {
          keys[(size_t)t * N + j0 + 32 + lane] = code1;
          if (ranks) pr1 = (uint32_t)atomicAdd(cnt + code1, 1);
          else atomicAdd(cnt + code1, 1);
        }
      }
      if (pend) {
        ranks[pidx] = pr0;
        if (pend1) ranks[pidx + 32] = pr1;
      }
    }
  }
}

// Counting as a pass of its own, for tables whose counters do not fit the L2 cache together (2^21 buckets x 64 tables
// are half a gigabyte): the blocks walk table after table, so that the counters being incremented at any moment are
// those of one or two tables and the atomics stay in L2.  ranks[t][j] = arrivals before j in its bucket.
__global__ void __launch_bounds__(256) k_count_ranks(const uint32_t* keys, uint32_t* ranks, int32_t* counts, int N, long long nb) {
  const int t = blockIdx.y;
  const uint32_t* k = keys + (size_t)t * N;
  uint32_t* r = ranks ? ranks + (size_t)t * N : nullptr;
  int32_t* cnt = counts + (size_t)t * (size_t)(nb + 1) + 1;
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < N; j += gridDim.x * blockDim.x) {
    const uint32_t v = (uint32_t)atomicAdd(cnt + k[j], 1);
    if (r) r[j] = v;
  }
}

// counts[t][0] = 0, counts[t][c + 1] = size of bucket c  ->  inclusive running sum = bucket offsets.
// Two kernels over chunks of BS_CHUNK counters: the sum of every chunk, then per chunk the sum of the
// table's earlier chunks plus a scan inside the chunk.
constexpr int ORD_SMALL = 16;     // buckets up to this size are put in order in registers
constexpr int ORD_BLOCK = 4096;   // up to this size by one block in shared memory
constexpr int BS_THREADS = 256;
constexpr int BS_PER = 16;
constexpr int BS_CHUNK = BS_THREADS * BS_PER;

__global__ void __launch_bounds__(BS_THREADS) k_bucket_sums(const int32_t* off, long long nb, int32_t* part, int nchunks) {
  __shared__ int sh[BS_THREADS / 32];
  const int32_t* o = off + (size_t)blockIdx.y * (size_t)(nb + 1);
  const long long n = nb + 1, base = (long long)blockIdx.x * BS_CHUNK;
  int sum = 0;
#pragma unroll
  for (int u = 0; u < BS_PER; ++u) {
    const long long i = base + threadIdx.x + (long long)u * BS_THREADS;
    sum += i < n ? o[i] : 0;
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    int tot = 0;
    for (int w = 0; w < BS_THREADS / 32; ++w) tot += sh[w];
    part[(size_t)blockIdx.y * nchunks + blockIdx.x] = tot;
  }
}

// With cnt != null the buckets of more than min_n (>= ORD_SMALL) ids are entered in the lists of the block-wide and
// the ordered-pass ordering kernels on the way (cnt[0] / cnt[1] are the lists' lengths).
__global__ void __launch_bounds__(BS_THREADS) k_bucket_scan(int32_t* off, long long nb, const int32_t* part, int nchunks,
                                                            int min_n, int2* mid, int2* big, int* cnt) {
  __shared__ int sh[BS_THREADS / 32 + 1];
  int32_t* o = off + (size_t)blockIdx.y * (size_t)(nb + 1);
  const long long n = nb + 1, base = (long long)blockIdx.x * BS_CHUNK;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // everything before this chunk
  int before = 0;
  for (int c = threadIdx.x; c < (int)blockIdx.x; c += BS_THREADS) before += part[(size_t)blockIdx.y * nchunks + c];
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) before += __shfl_xor_sync(0xffffffffu, before, d);
  if (lane == 0) sh[warp] = before;
  __syncthreads();
  before = 0;
  for (int w = 0; w < BS_THREADS / 32; ++w) before += sh[w];
  __syncthreads();
  // the chunk itself: every warp owns BS_PER * 32 consecutive counters and walks them 32 at a time
  const long long wbase = base + (long long)warp * (BS_PER * 32);
  int v[BS_PER];
  int wsum = 0;
#pragma unroll
  for (int u = 0; u < BS_PER; ++u) {
    const long long i = wbase + u * 32 + lane;
    v[u] = i < n ? o[i] : 0;
    wsum += v[u];
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) wsum += __shfl_xor_sync(0xffffffffu, wsum, d);
  if (lane == 0) sh[warp] = wsum;
  __syncthreads();
  int run = before;
  for (int w = 0; w < warp; ++w) run += sh[w];
#pragma unroll
  for (int u = 0; u < BS_PER; ++u) {
    int incl = v[u];
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      int x = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += x;
    }
    const long long i = wbase + u * 32 + lane;
    if (i < n) o[i] = run + incl;
    if (cnt && i >= 1 && i < n && v[u] > min_n) {          // word i counts bucket i - 1
      if (v[u] <= ORD_BLOCK) mid[atomicAdd(cnt, 1)] = make_int2((int)blockIdx.y, (int)(i - 1));
      else big[atomicAdd(cnt + 1, 1)] = make_int2((int)blockIdx.y, (int)(i - 1));
    }
    run += __shfl_sync(0xffffffffu, incl, 31);
  }
}

// ------------------------------------------------------------------ stable LSD radix sort, per table
constexpr int SORT_THREADS = 512;
constexpr int SORT_WARPS = SORT_THREADS / 32;
constexpr int SORT_TILE = 8192;                      // elements per block
constexpr int SORT_SUB = SORT_TILE / SORT_WARPS;     // contiguous elements per warp
constexpr int SORT_ITERS = SORT_SUB / 32;            // groups of 32 keys a warp walks, all fetched up front
constexpr int SORT_MAX_WIDTH = 9;                    // bits per pass

// hist[t][digit][tile] = number of keys of that digit in the tile.
__global__ void __launch_bounds__(SORT_THREADS)
k_sort_hist(const uint32_t* keys, int32_t* hist, int N, int tiles, int shift, int width) {
  __shared__ int cnt[1 << SORT_MAX_WIDTH];
  const int radix = 1 << width, t = blockIdx.y, tl = blockIdx.x;
  for (int d = threadIdx.x; d < radix; d += SORT_THREADS) cnt[d] = 0;
  __syncthreads();
  const uint32_t* k = keys + (size_t)t * N;
  const int beg = tl * SORT_TILE, end = min(N, beg + SORT_TILE);
  for (int i = beg + threadIdx.x; i < end; i += SORT_THREADS) atomicAdd(&cnt[(k[i] >> shift) & (radix - 1)], 1);
  __syncthreads();
  for (int d = threadIdx.x; d < radix; d += SORT_THREADS) hist[((size_t)t * radix + d) * tiles + tl] = cnt[d];
}

// Exclusive scan of hist[t][*][*] in (digit, tile) order: where each tile's run of each digit starts.
__global__ void __launch_bounds__(1024) k_sort_scan(int32_t* hist, int n) {
  __shared__ int sh[33];
  int32_t* o = hist + (size_t)blockIdx.x * n;
  const int chunk = (n + 1023) / 1024;
  const int beg = min(n, (int)threadIdx.x * chunk), end = min(n, beg + chunk);
  int sum = 0;
  for (int i = beg; i < end; ++i) sum += o[i];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = sum;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    int v = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += v;
  }
  if (lane == 31) sh[warp] = incl;
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = 0;
    for (int w = 0; w < 32; ++w) { int c = sh[w]; sh[w] = run; run += c; }
  }
  __syncthreads();
  int run = incl - sum + sh[warp];
  for (int i = beg; i < end; ++i) { int c = o[i]; o[i] = run; run += c; }
}

// Each warp owns a contiguous part of the tile and walks it in order, 32 keys at a time; equal
// digits inside a group of 32 are ranked by lane with a match mask, so the order of equal digits is
// kept.  All of a warp's keys (and values) are fetched before the walk.  The walk places the elements
// in shared memory in digit order; they are then written out in that order, so that a warp's stores
// cover a few contiguous runs instead of 32 scattered words.
// vals_in == nullptr means the value of element i is i (first pass).  keys_out may be nullptr
// (last pass).
constexpr int SORT_RADIX_MAX = 1 << SORT_MAX_WIDTH;
constexpr int SORT_SMEM = (2 * SORT_TILE + SORT_WARPS * SORT_RADIX_MAX + 2 * SORT_RADIX_MAX + 64) * 4;

__global__ void __launch_bounds__(SORT_THREADS, 2)
k_sort_scatter(const uint32_t* keys_in, const int32_t* vals_in, uint32_t* keys_out, int32_t* vals_out,
               const int32_t* hist, int N, int tiles, int shift, int width) {
  extern __shared__ __align__(16) int ss_smem[];
  uint32_t* skey = reinterpret_cast<uint32_t*>(ss_smem);                 // [SORT_TILE] the tile in digit order
  int* sval = ss_smem + SORT_TILE;                                       // [SORT_TILE]
  int* offs = ss_smem + 2 * SORT_TILE;                                   // [SORT_WARPS][radix] cursor of (warp, digit) in the tile
  int* gbase = offs + SORT_WARPS * SORT_RADIX_MAX;                       // [radix] where the tile's run of a digit starts globally
  int* tbase = gbase + SORT_RADIX_MAX;                                   // [radix] where it starts inside the tile
  int* sh = tbase + SORT_RADIX_MAX;                                      // [33] scan scratch
  const int radix = 1 << width, t = blockIdx.y, tl = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t* kin = keys_in + (size_t)t * N;
  const int32_t* vin = vals_in ? vals_in + (size_t)t * N : nullptr;
  uint32_t* kout = keys_out ? keys_out + (size_t)t * N : nullptr;
  int32_t* vout = vals_out + (size_t)t * N;
  const int tbeg = tl * SORT_TILE, tn = min(SORT_TILE, N - tbeg);
  const int wbeg = min(N, tbeg + warp * SORT_SUB), wend = min(N, wbeg + SORT_SUB);

  uint32_t key[SORT_ITERS];
#pragma unroll
  for (int it = 0; it < SORT_ITERS; ++it) {
    const int i = wbeg + it * 32 + lane;
    key[it] = i < wend ? kin[i] : 0u;
  }
  int* myoffs = offs + warp * SORT_RADIX_MAX;
  for (int d = lane; d < radix; d += 32) myoffs[d] = 0;
  __syncwarp();
  // walk 1: rank of every element among the warp's elements of the same digit (counts fall out at the end)
  unsigned short lrank[SORT_ITERS];
#pragma unroll
  for (int it = 0; it < SORT_ITERS; ++it) {
    const bool live = wbeg + it * 32 + lane < wend;
    const int digit = live ? (int)((key[it] >> shift) & (radix - 1)) : radix + lane;   // dead lanes match nobody
    const unsigned peers = __match_any_sync(0xffffffffu, digit);
    const int rank = __popc(peers & ((1u << lane) - 1u));
    int base = 0;
    if (live) base = myoffs[digit];
    __syncwarp();
    if (live && rank == 0) myoffs[digit] = base + __popc(peers);
    __syncwarp();
    lrank[it] = (unsigned short)(base + rank);
  }
  __syncthreads();
  // per digit: the tile's count, the warps' starts relative to the digit's run, the global start of the run
  int cnt[(SORT_RADIX_MAX + SORT_THREADS - 1) / SORT_THREADS];
#pragma unroll
  for (int u = 0; u < (SORT_RADIX_MAX + SORT_THREADS - 1) / SORT_THREADS; ++u) {
    const int d = threadIdx.x + u * SORT_THREADS;
    cnt[u] = 0;
    if (d < radix) {
      int run = 0;
      for (int w = 0; w < SORT_WARPS; ++w) { int c = offs[w * SORT_RADIX_MAX + d]; offs[w * SORT_RADIX_MAX + d] = run; run += c; }
      cnt[u] = run;
      gbase[d] = hist[((size_t)t * radix + d) * tiles + tl];
    }
  }
  // exclusive scan of the counts over the digits (digit d lives in thread d % SORT_THREADS, round d / SORT_THREADS)
  int carry = 0;
#pragma unroll
  for (int u = 0; u < (SORT_RADIX_MAX + SORT_THREADS - 1) / SORT_THREADS; ++u) {
    int incl = cnt[u];
#pragma unroll
    for (int dd = 1; dd < 32; dd <<= 1) {
      int x = __shfl_up_sync(0xffffffffu, incl, dd);
      if (lane >= dd) incl += x;
    }
    __syncthreads();
    if (lane == 31) sh[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int w = lane < SORT_WARPS ? sh[lane] : 0, wi = w;
#pragma unroll
      for (int dd = 1; dd < 32; dd <<= 1) {
        int x = __shfl_up_sync(0xffffffffu, wi, dd);
        if (lane >= dd) wi += x;
      }
      if (lane < SORT_WARPS) sh[lane] = wi - w;
      if (lane == 31) sh[32] = wi;
    }
    __syncthreads();
    const int d = threadIdx.x + u * SORT_THREADS;
    if (d < radix) tbase[d] = carry + sh[warp] + incl - cnt[u];
    carry += sh[32];
  }
  __syncthreads();
  // walk 2: place the elements in digit order in shared memory
#pragma unroll
  for (int it = 0; it < SORT_ITERS; ++it) {
    const int i = wbeg + it * 32 + lane;
    if (i < wend) {
      const int digit = (int)((key[it] >> shift) & (radix - 1));
      const int lpos = tbase[digit] + myoffs[digit] + (int)lrank[it];
      skey[lpos] = key[it];
      sval[lpos] = vin ? vin[i] : i;
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < tn; i += SORT_THREADS) {
    const uint32_t k = skey[i];
    const int d = (int)((k >> shift) & (radix - 1));
    const int g = gbase[d] + (i - tbase[d]);
    if (kout) kout[g] = k;
    vout[g] = sval[i];
  }
}

// ------------------------------------------------------------------ wide codes: place, then order inside buckets
// With codes wider than one radix digit the buckets are small (a few ids on average), and sorting the whole table
// twice is a detour.  Instead the hashing kernel's counting atomics hand every id its rank of arrival inside its
// bucket, the id goes to the bucket's start plus that rank, and the ids of each bucket are then put in ascending
// order where they stand: in registers for
// buckets of up to ORD_SMALL ids, by a block-wide sort in shared memory up to ORD_BLOCK, and for a larger bucket by
// one ordered pass over the table's codes that writes the matching ids out again.
constexpr int ORD_THREADS = 256;

__global__ void __launch_bounds__(256) k_place_ids(const uint32_t* keys, const uint32_t* ranks, const int32_t* off, int32_t* ids,
                                                   int N, long long nb) {
  const int t = blockIdx.y;
  const uint32_t* k = keys + (size_t)t * N;
  const uint32_t* r = ranks + (size_t)t * N;
  const int32_t* o = off + (size_t)t * (size_t)(nb + 1);
  int32_t* out = ids + (size_t)t * N;
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < N; j += gridDim.x * blockDim.x)
    out[__ldg(o + k[j]) + (int)r[j]] = j;
}

// Sorts n <= M ids in place with an odd-even transposition network (fully unrolled: the ids stay in registers).
template <int M>
__device__ __forceinline__ void order_in_registers(int32_t* p, int n) {
  int a[M];
#pragma unroll
  for (int i = 0; i < M; ++i) a[i] = i < n ? p[i] : 0x7fffffff;
#pragma unroll
  for (int round = 0; round < M; ++round) {
#pragma unroll
    for (int i = round & 1; i + 1 < M; i += 2) {
      const int lo = min(a[i], a[i + 1]), hi = max(a[i], a[i + 1]);
      a[i] = lo; a[i + 1] = hi;
    }
  }
#pragma unroll
  for (int i = 0; i < M; ++i)
    if (i < n) p[i] = a[i];
}

// One thread per bucket.  cnt[0] / cnt[1]: lengths of the lists of buckets left to the block-wide and to the ordered-
// pass kernels.
// Only buckets of more than min_n ids are touched.
__global__ void __launch_bounds__(256) k_order_small(const int32_t* off, int32_t* ids, int N, long long nb, int2* mid,
                                                     int2* big, int* cnt, int min_n) {
  const int t = blockIdx.y;
  const int32_t* o = off + (size_t)t * (size_t)(nb + 1);
  int32_t* out = ids + (size_t)t * N;
  for (long long c = (long long)blockIdx.x * blockDim.x + threadIdx.x; c < nb; c += (long long)gridDim.x * blockDim.x) {
    const int beg = o[c], n = o[c + 1] - beg;
    if (n <= min_n) continue;
    if (n <= 4) order_in_registers<4>(out + beg, n);
    else if (n <= 8) order_in_registers<8>(out + beg, n);
    else if (n <= ORD_SMALL) order_in_registers<ORD_SMALL>(out + beg, n);
    else if (n <= ORD_BLOCK) {
      mid[atomicAdd(cnt, 1)] = make_int2(t, (int)c);
    } else {
      big[atomicAdd(cnt + 1, 1)] = make_int2(t, (int)c);
    }
  }
}

// Buckets of ORD_SMALL + 1 .. ORD_BLOCK ids: a block loads one, sorts it in shared memory (bitonic) and writes it back.
__global__ void __launch_bounds__(ORD_THREADS) k_order_mid(const int32_t* off, int32_t* ids, int N, long long nb, const int2* mid,
                                                           const int* cnt) {
  __shared__ int sm[ORD_BLOCK];
  const int nmid = cnt[0];
  for (int q = blockIdx.x; q < nmid; q += gridDim.x) {
    const int2 tc = mid[q];
    const int32_t* o = off + (size_t)tc.x * (size_t)(nb + 1);
    int32_t* out = ids + (size_t)tc.x * N;
    const int beg = o[tc.y], n = o[tc.y + 1] - beg;
    int n2 = 1;
    while (n2 < n) n2 <<= 1;
    __syncthreads();
    for (int i = threadIdx.x; i < n2; i += ORD_THREADS) sm[i] = i < n ? out[beg + i] : 0x7fffffff;
    __syncthreads();
    for (int k = 2; k <= n2; k <<= 1)
      for (int j = k >> 1; j > 0; j >>= 1) {
        for (int i = threadIdx.x; i < n2; i += ORD_THREADS) {
          const int x = i ^ j;
          if (x > i) {
            const int a = sm[i], b = sm[x];
            const bool asc = (i & k) == 0;
            if ((a > b) == asc) { sm[i] = b; sm[x] = a; }
          }
        }
        __syncthreads();
      }
    for (int i = threadIdx.x; i < n; i += ORD_THREADS) out[beg + i] = sm[i];
  }
}

// Larger buckets: the ids of bucket c in ascending order are the j, ascending, whose code is c.
__global__ void __launch_bounds__(ORD_THREADS) k_order_big(const uint32_t* keys, const int32_t* off, int32_t* ids, int N,
                                                           long long nb, const int2* big, const int* cnt) {
  __shared__ int sh[ORD_THREADS / 32 + 1];
  const int nbig = cnt[1];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int q = blockIdx.x; q < nbig; q += gridDim.x) {
    const int2 tc = big[q];
    const uint32_t* k = keys + (size_t)tc.x * N;
    int32_t* out = ids + (size_t)tc.x * N + off[(size_t)tc.x * (size_t)(nb + 1) + tc.y];
    int run = 0;
    for (int base = 0; base < N; base += ORD_THREADS) {
      const int j = base + threadIdx.x;
      const bool hit = j < N && k[j] == (uint32_t)tc.y;
      const unsigned m = __ballot_sync(0xffffffffu, hit);
      __syncthreads();
      if (lane == 0) sh[warp] = __popc(m);
      __syncthreads();
      int before = 0, total = 0;
      for (int w = 0; w < ORD_THREADS / 32; ++w) { const int x = sh[w]; if (w < warp) before += x; total += x; }
      if (hit) out[run + before + __popc(m & ((1u << lane) - 1u))] = j;
      run += total;
    }
  }
}

// Puts the ids of every bucket with more than min_n ids in ascending order (place path only).  With `listed`, the
// offset scan has already entered those buckets in the lists (all of them larger than ORD_SMALL).
static cudaError_t order_buckets(Ctx* c, int min_n, bool listed) {
  if (min_n < 1) min_n = 1;
  LaunchScope ls(c, KID_ORDER_BUCKETS);
  if (!listed) {
    cudaError_t e = cudaMemsetAsync(c->ord_cnt, 0, 2 * sizeof(int), c->stream);
    if (e != cudaSuccess) return e;
    dim3 grid((unsigned)min((long long)((c->nb + 255) / 256), 2048LL), c->L);
    k_order_small<<<grid, 256, 0, c->stream>>>(c->bucket_off, c->bucket_ids, c->N, c->nb, c->ord_mid, c->ord_big, c->ord_cnt, min_n);
  }
  k_order_mid<<<c->num_sms * 4, ORD_THREADS, 0, c->stream>>>(c->bucket_off, c->bucket_ids, c->N, c->nb, c->ord_mid, c->ord_cnt);
  k_order_big<<<c->num_sms, ORD_THREADS, 0, c->stream>>>(c->keysA, c->bucket_off, c->bucket_ids, c->N, c->nb, c->ord_big,
                                                          c->ord_cnt);
  return cudaGetLastError();
}

cudaError_t launch_order_buckets(Ctx* c, int min_n) { return order_buckets(c, min_n, false); }

cudaError_t launch_build_tables(Ctx* c) {
  const size_t off_bytes = (size_t)c->L * (size_t)(c->nb + 1) * sizeof(int32_t);
  cudaError_t e = cudaMemsetAsync(c->bucket_off, 0, off_bytes, c->stream);
  if (e != cudaSuccess) return e;
  // the counting atomics ride with the hashing while all the tables' counters fit the L2 cache together; beyond that
  // every atomic would be a read-modify-write in DRAM, and the counting becomes a pass of its own, table by table
  const bool split_count = off_bytes > COUNT_SPLIT_BYTES;
  int32_t* hash_counts = split_count ? nullptr : c->bucket_off;
  const int tile_bytes = (HN_ROWS * (c->H + 1) * (int)sizeof(float) + 15) & ~15;
  const long long fn_bytes = (long long)c->KL * c->fn_len * 2;
  const bool fn_smem = fn_bytes <= HN_FN_SMEM_MAX && c->H <= 0x7fff;
  const int smem = tile_bytes + (fn_smem ? (int)fn_bytes : 0);
  const long long smem2_ll = ((32LL * (c->H + 1) * 8 + 15) & ~15LL) + fn_bytes;
  if (fn_smem && c->cfg.hash_family == DSLIDE_DWTA && c->fn_len == 8 && smem2_ll <= 100 * 1024) {
    const int smem2 = (int)smem2_ll;
    if (smem2 > 48 * 1024) {
      e = cudaFuncSetAttribute(split_count ? k_hash_neurons_dwta8<false> : k_hash_neurons_dwta8<true>,
                               cudaFuncAttributeMaxDynamicSharedMemorySize, smem2);
      if (e != cudaSuccess) return e;
    }
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, split_count ? k_hash_neurons_dwta8<false> : k_hash_neurons_dwta8<true>,
                                                      HN_THREADS, smem2);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    LaunchScope ls(c, KID_HASH_NEURONS);
    auto kern8 = split_count ? k_hash_neurons_dwta8<false> : k_hash_neurons_dwta8<true>;
    kern8<<<c->num_sms * per_sm, HN_THREADS, smem2, c->stream>>>(c->W2, c->hash_idx, c->keysA, c->place_path ? c->keysB : nullptr,
                                                               hash_counts, c->N, c->H, c->K, c->L, c->lg_bin, c->nb);
  } else {
    auto kern = fn_smem ? k_hash_neurons<true> : k_hash_neurons<false>;
    if (smem > 48 * 1024) {
      e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      if (e != cudaSuccess) return e;
    }
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, HN_THREADS, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    LaunchScope ls(c, KID_HASH_NEURONS);
    kern<<<c->num_sms * per_sm, HN_THREADS, smem, c->stream>>>(c->W2, c->hash_idx, c->hash_sign, c->keysA,
                                                             c->place_path ? c->keysB : nullptr, hash_counts, c->N, c->H, c->K, c->L,
                                                             c->cfg.hash_family, c->lg_bin, c->fn_len, c->nb);
  }
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  if (split_count) {
    LaunchScope ls(c, KID_HASH_NEURONS);
    dim3 grid((unsigned)min((long long)(c->N + 255) / 256, 2048LL), c->L);
    k_count_ranks<<<grid, 256, 0, c->stream>>>(c->keysA, c->place_path ? c->keysB : nullptr, c->bucket_off, c->N, c->nb);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  const bool list_in_scan = c->place_path && c->cap >= ORD_SMALL;
  {
    const int nchunks = (int)((c->nb + 1 + BS_CHUNK - 1) / BS_CHUNK);
    dim3 grid(nchunks, c->L);
    // on the place path, with a cap of at least ORD_SMALL, the buckets that must be in order for the step (those
    // above the cap) are listed by the scan itself: no separate pass over all bucket sizes
    if (list_in_scan && (e = cudaMemsetAsync(c->ord_cnt, 0, 2 * sizeof(int), c->stream)) != cudaSuccess) return e;
    LaunchScope ls(c, KID_BUCKET_SCAN);
    k_bucket_sums<<<grid, BS_THREADS, 0, c->stream>>>(c->bucket_off, c->nb, c->bucket_part, nchunks);
    k_bucket_scan<<<grid, BS_THREADS, 0, c->stream>>>(c->bucket_off, c->nb, c->bucket_part, nchunks, c->cap, c->ord_mid,
                                                      c->ord_big, list_in_scan ? c->ord_cnt : nullptr);
  }
  if ((e = cudaGetLastError()) != cudaSuccess) return e;

  if (c->place_path) {
    {
      LaunchScope ls(c, KID_PLACE_IDS);
      dim3 grid((unsigned)min((long long)(c->N + 255) / 256, 1024LL), c->L);
      k_place_ids<<<grid, 256, 0, c->stream>>>(c->keysA, c->keysB, c->bucket_off, c->bucket_ids, c->N, c->nb);
    }
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    // A query reads a whole bucket unless it holds more than `cap` ids, and the union of the buckets is put in
    // order afterwards anyway: only buckets larger than the cap must be in ascending order for the step.  The
    // smaller ones are ordered when the table is read back (launch_order_buckets(c, 1)).
    c->ids_ordered_above = c->cap;
    return order_buckets(c, c->cap, list_in_scan);
  }

  if ((e = cudaFuncSetAttribute(k_sort_scatter, cudaFuncAttributeMaxDynamicSharedMemorySize, SORT_SMEM)) != cudaSuccess) return e;
  const uint32_t* kin = c->keysA;
  const int32_t* vin = nullptr;
  for (int pass = 0; pass < c->sort_passes; ++pass) {
    const bool last = pass == c->sort_passes - 1;
    const int shift = pass * c->sort_width;
    const int width = min(c->sort_width, c->bits - shift);
    const int radix = 1 << width;
    uint32_t* kout = last ? nullptr : (kin == c->keysA ? c->keysB : c->keysA);
    int32_t* vout = last ? c->bucket_ids : (vin == c->valsA ? c->valsB : c->valsA);
    dim3 grid(c->sort_tiles, c->L);
    {
      LaunchScope ls(c, KID_SORT_HIST);
      k_sort_hist<<<grid, SORT_THREADS, 0, c->stream>>>(kin, c->tile_hist, c->N, c->sort_tiles, shift, width);
    }
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    {
      LaunchScope ls(c, KID_SORT_SCAN);
      k_sort_scan<<<c->L, 1024, 0, c->stream>>>(c->tile_hist, radix * c->sort_tiles);
    }
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    {
      LaunchScope ls(c, KID_SORT_SCATTER);
      k_sort_scatter<<<grid, SORT_THREADS, SORT_SMEM, c->stream>>>(kin, vin, kout, vout, c->tile_hist, c->N, c->sort_tiles,
                                                          shift, width);
    }
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    kin = kout;
    vin = vout;
  }
  return cudaSuccess;
}

int sort_tile_elems() { return SORT_TILE; }
int order_small_max() { return ORD_SMALL; }
int order_block_max() { return ORD_BLOCK; }
int bucket_scan_chunk() { return BS_CHUNK; }
int sort_max_width() { return SORT_MAX_WIDTH; }

}  // namespace dslide
