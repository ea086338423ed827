// Inference over all N neurons on the tensor pipe (dslide_predict_topk with dense = 1, k <= TC_K_MAX).
//
// The logits of a batch against every output neuron are one contraction, Z[B][N] = h[B][H] . W2[N][H]^T + b2
// (Section 3.6: "layer sparsity is 1"), so this path runs it on the fifth-generation tensor cores: tiles of W2
// arrive in shared memory by TMA (cp.async.bulk.tensor, 128-byte swizzle), the 128 samples' hidden activations of a
// block sit in tensor memory beside the accumulators, a single thread issues tcgen05.mma (kind::tf32), and the
// read-back warps fetch the accumulators (tcgen05.ld) and keep, per sample, the candidates of the block's slice of
// neurons; one more warp takes the largest row norm of W2 from the tiles while they are in shared memory.  W2 is
// streamed once per 128 samples (the groups of samples walk the same tiles together, so HBM sees it once per call).
//
// TF32 rounds both operands to 10 mantissa bits, far from the 1e-4 the scores must meet.  The tensor pass is
// therefore a FILTER, in two launches of the same kernel.  The first scores every TC_SUBSET-th tile of neurons and
// writes the scores out; k_tc_tau takes, per sample, about the cap-th best of them (cap = 2k + TC_EXTRA) as the
// sample's threshold -- about cap * TC_SUBSET neurons reach it over all N.  The second launch scores all tiles and a
// thread appends the few scores of its sample that reach the threshold to the sample's candidate buffer.
// k_tc_refine recomputes the cap or so best candidates exactly in fp32 and orders them (logit descending, id
// ascending).  The filter is exact when the k-th exact score clears every discarded neuron's approximate score by
// more than the approximation's error bound, 2^-9 |h| |w|_max (plus accumulation); a sample for which that cannot
// be shown (or whose buffers ran over) is flagged and its block then scores all N neurons for it in fp32.  Results
// are therefore those of the exact path.  The kernels of a call follow one another by programmatic dependent launch.
#include <cuda.h>

#include "common.cuh"

namespace dslide {

constexpr int TC_M = 128;          // samples per block = lanes of the accumulator
constexpr int TC_N = 128;          // neurons per tile = columns of the accumulator
constexpr int TC_KB = 32;          // hidden units per 128-byte swizzled row
constexpr int TC_STAGES = 3;       // tiles of W2 in flight at most (as many as fit in shared memory)
constexpr int TC_NACC = 3;         // tensor memory: up to three accumulators of TC_N columns (two when H > TC_N), then the activations (H columns)
constexpr int TC_TMEM_COLS = 512;
constexpr int TC_SPLIT = 4;        // read-back warps per quarter of tensor memory (each takes 1 / TC_SPLIT of a tile's columns)
constexpr int TC_EPI = 128 * TC_SPLIT;                 // read-back threads
constexpr int TC_THREADS = 96 + TC_EPI;                // warp 0: TMA producer; warp 1: tensor memory + MMA issue; warp 2: row norms; then the read-back warps
constexpr int TC_EXTRA = 8;        // candidates kept beyond k: TC_EXTRA + k (the wider the margin, the rarer the exact fall-back)
constexpr int TC_K_MAX = 8;
constexpr int TC_GBUF_MIN = 64;    // candidate slots per (buffer, sample) at least; a buffer that runs over sends the sample to the exact scan
constexpr int TC_TARGET = 64;      // candidates aimed at per sample: TC_TARGET x cap
constexpr int TC_SUBSET = 64;      // the threshold pass scores every TC_SUBSET-th tile
constexpr int TC_SUB_BYTES = TC_M * 128;               // one 32-unit slab of 128 rows
constexpr float TC_ERR = 2.2e-3f;  // |approximate - exact| <= TC_ERR * |h| * |w|: two operands cut to 10 mantissa bits, fp32 sums

struct TcParams {
  const RowHdr* hdr2;
  const float* h;                  // [>= B][H] hidden activations of the batch
  int2* cand;                      // [TC_SPLIT * slices][Bpad][gbuf] (score bits, id), cand_cnt of them valid, no order
  int* cand_cnt;                   // [TC_SPLIT * slices][Bpad]
  float* dump;                     // DUMP launch: [Bpad][dump_cols] scores of the subset's tiles
  const float* tau;                // filter launch: [Bpad] thresholds
  int* need_fix;                   // [B] set when a sample's buffer ran over
  unsigned int* norm2max;          // filter launch: largest squared norm of a row of W2, as the bits of a non-negative float
  DevState* st;
  int B, Bpad, H, N, nslices, ntiles;          // ntiles: tiles this launch walks
  int tile_stride;                 // tile i of the launch is tile i * tile_stride of W2
  int stages;                      // tiles of W2 in flight, 1 .. TC_STAGES
  int dump_cols;
  int gbuf;                        // slots per candidate buffer
};

__device__ __forceinline__ uint32_t tc_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void tc_bar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(tc_smem(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void tc_bar_expect(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(tc_smem(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tc_bar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(tc_smem(bar)) : "memory");
}
// Bounded wait; once any wait of the block has run out, *abort is set and every later wait returns at once, so that
// all the roles run through their loops, tensor memory is released and the kernel ends (its results are flagged).
__device__ __forceinline__ void tc_bar_wait(uint64_t* bar, uint32_t parity, volatile int* abort) {
  const uint32_t a = tc_smem(bar);
  for (int it = 0; it < (1 << 20); ++it) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(a), "r"(parity), "r"(2000u) : "memory");      // may sleep up to 2 us per try: a waiting warp issues little
    if (ok) return;
    if ((it & 1023) == 1023 && *abort) return;
  }
  *abort = 1;
}
__device__ __forceinline__ void tc_tma_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(tc_smem(dst)), "l"(map), "r"(x), "r"(y), "r"(tc_smem(bar)) : "memory");
}
// Shared-memory operand descriptor: K-major tile of 128-byte rows, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t tc_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);            // start address
  d |= (uint64_t)1 << 16;                              // leading-dimension offset: unused with swizzled K-major rows
  d |= (uint64_t)(1024 >> 4) << 32;                    // stride between groups of eight rows
  d |= (uint64_t)1 << 46;                              // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                              // 128-byte swizzle
  return d;
}
// Instruction descriptor: fp32 accumulator, tf32 x tf32, both operands K-major, N x M tile.
__host__ __device__ constexpr uint32_t tc_idesc(int M, int N) {
  return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// D[tmem] (+)= A[tmem] . B[smem]^T: the first operand is read from tensor memory, so shared memory serves one operand only
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint32_t a_tmem, uint64_t b, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
               ::"r"(d_tmem), "r"(a_tmem), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, "
      "%19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
        "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
        "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(tc_smem(bar)) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, "
      "%19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ bool tc_better(float za, int ia, float zb, int ib) { return za > zb || (za == zb && ia < ib); }

// Grid: (slices of the neurons, groups of 128 samples).  Dynamic shared memory (1024-byte aligned):
// TC_STAGES tiles of W2 as [H/32][128 rows][128 B], then
// the tiles' biases, the barriers.  (The samples' candidate buffers are in global memory.)
template <bool DUMP>      // DUMP: write every score out (threshold pass); else append the scores that reach the sample's threshold
__global__ void __launch_bounds__(TC_THREADS, 1)
k_dense_tc(const __grid_constant__ CUtensorMap tmW, const TcParams p) {
  extern __shared__ __align__(1024) unsigned char tc_smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~(uintptr_t)1023);
  const int ksub = p.H / TC_KB;
  const uint32_t tile_bytes = (uint32_t)ksub * TC_SUB_BYTES;
  unsigned char* smB = sm;
  const int nst = p.stages;
  float* sb = reinterpret_cast<float*>(smB + (size_t)nst * tile_bytes);                         // [accumulator][128] biases of its tile
  uint64_t* bars = reinterpret_cast<uint64_t*>(sb + TC_NACC * TC_N);
  uint64_t* bar_a = bars;                      // activations are in tensor memory
  uint64_t* bar_full = bars + 1;               // [TC_STAGES] tile of W2 has arrived
  uint64_t* bar_empty = bars + 1 + TC_STAGES;  // [TC_STAGES] tile of W2 has been consumed
  uint64_t* bar_accfull = bars + 1 + 2 * TC_STAGES;              // [TC_NACC] accumulator written
  uint64_t* bar_accempty = bars + 1 + 2 * TC_STAGES + TC_NACC;   // [TC_NACC] accumulator read back
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 1 + 2 * TC_STAGES + 2 * TC_NACC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int slice = blockIdx.x, s0 = blockIdx.y * TC_M;
  // tiles of this slice: slice, slice + nslices, ... (both sample groups walk the same tiles at the same time: the
  // second read of a tile is served by L2)
  const int my_tiles = slice < p.ntiles ? (p.ntiles - slice + p.nslices - 1) / p.nslices : 0;
  // The filter launch also takes the largest squared row norm of W2 (the error bound needs it) from the tiles as
  // they pass through shared memory; up to four sample groups share a tile's rows (they all see the same tiles).
  const int nshare = gridDim.y >= 4 ? 4 : (gridDim.y >= 2 ? 2 : 1);      // blocks that share a tile's 128 rows
  const bool norms = !DUMP && (int)blockIdx.y < nshare;
  const int nacc = p.H <= TC_N ? TC_NACC : 2;      // accumulators in use; the activations follow them
  const uint32_t acol = (uint32_t)(nacc * TC_N);

  if (tid == 0) {
    tc_bar_init(bar_a, 128);
    for (int i = 0; i < TC_STAGES; ++i) { tc_bar_init(bar_full + i, 1); tc_bar_init(bar_empty + i, norms ? 2 : 1); }
    for (int i = 0; i < TC_NACC; ++i) { tc_bar_init(bar_accfull + i, 1); tc_bar_init(bar_accempty + i, TC_EPI); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {      // tensor memory: all of it (one block per SM)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem(tmem_slot)), "r"(TC_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  griddep_launch_dependents();       // the next kernel of the call may be placed as blocks of this one leave
  griddep_wait();                    // the filter launch reads the thresholds of the kernel before it

  if (warp == 0) {
    // ---------------- producer: one thread feeds the TMA ----------------
    if (lane == 0) {
      int st = 0, stround = 0;
      for (int i = 0; i < my_tiles; ++i) {
        if (stround > 0) tc_bar_wait(bar_empty + st, (stround - 1) & 1, abort_flag);
        const int row0 = (slice + i * p.nslices) * p.tile_stride * TC_N;
        tc_bar_expect(bar_full + st, tile_bytes);
        for (int ks = 0; ks < ksub; ++ks)
          tc_tma_2d(smB + (size_t)st * tile_bytes + (size_t)ks * TC_SUB_BYTES, &tmW, ks * TC_KB, row0, bar_full + st);
        if (++st == nst) { st = 0; ++stround; }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issue: one thread ----------------
    if (lane == 0) {
      const uint32_t idesc = tc_idesc(TC_M, TC_N);
      tc_bar_wait(bar_a, 0, abort_flag);
      const uint64_t b_base = tc_desc(tc_smem(smB));      // a descriptor's address field counts 16-byte units
      int st = 0, stround = 0, acc = 0, accround = 0;
      for (int i = 0; i < my_tiles; ++i) {
        tc_bar_wait(bar_full + st, stround & 1, abort_flag);
        if (accround > 0) tc_bar_wait(bar_accempty + acc, (accround - 1) & 1, abort_flag);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d = tmem_base + (uint32_t)(acc * TC_N);
        const uint64_t b_tile = b_base + (uint64_t)(((uint32_t)st * tile_bytes) >> 4);
        for (int ks = 0; ks < ksub; ++ks) {
          const uint32_t a = tmem_base + acol + (uint32_t)(ks * TC_KB);      // lanes = samples, columns = hidden units
          const uint64_t b = b_tile + (uint64_t)((ks * TC_SUB_BYTES) >> 4);
#pragma unroll
          for (int kk = 0; kk < TC_KB / 8; ++kk)              // eight tf32 = 32 bytes per instruction
            tc_mma(d, a + (uint32_t)(kk * 8), b + (uint64_t)(kk * 2), idesc, (ks | kk) != 0 ? 1u : 0u);
        }
        tc_commit(bar_empty + st);          // the tile's shared memory is free once these instructions have read it
        tc_commit(bar_accfull + acc);       // and the accumulator is complete
        if (++st == nst) { st = 0; ++stround; }
        if (++acc == nacc) { acc = 0; ++accround; }
      }
    }
  } else if (warp == 2) {
    // ---------------- row norms: lane = row modulo 32; sums of squares do not care about the swizzle, but the
    // lanes of a quarter-warp read different 16-byte pieces so that all banks are busy ----------------
    if (norms) {
      float best = 0.f;
      int st = 0, stround = 0;
      for (int i = 0; i < my_tiles; ++i) {
        tc_bar_wait(bar_full + st, stround & 1, abort_flag);
        const unsigned char* tile = smB + (size_t)st * tile_bytes;
        const int nrr = 4 / nshare;                    // rows of this block: nrr per lane
        for (int rr = 0; rr < nrr; ++rr) {
          const unsigned char* rowp = tile + (size_t)(32 * (nrr * (int)blockIdx.y + rr) + lane) * 128;
          unsigned long long s0 = 0ull, s1 = 0ull;    // two pairs of partial sums (packed fp32 fused multiply-adds)
          for (int ks = 0; ks < ksub; ++ks)
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              const ulonglong2 w = *reinterpret_cast<const ulonglong2*>(rowp + (size_t)ks * TC_SUB_BYTES + (size_t)((c ^ (lane & 7)) * 16));
              asm("fma.rn.f32x2 %0, %1, %1, %0;" : "+l"(s0) : "l"(w.x));
              asm("fma.rn.f32x2 %0, %1, %1, %0;" : "+l"(s1) : "l"(w.y));
            }
          const float ssum = (__uint_as_float((unsigned)s0) + __uint_as_float((unsigned)(s0 >> 32))) +
                             (__uint_as_float((unsigned)s1) + __uint_as_float((unsigned)(s1 >> 32)));
          best = fmaxf(best, ssum);
        }
        __syncwarp();
        if (lane == 0) tc_bar_arrive(bar_empty + st);
        if (++st == nst) { st = 0; ++stround; }
      }
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, d));
      if (lane == 0) atomicMax(p.norm2max, __float_as_uint(best));
    }
  } else {
    // ---------------- read-back: thread = (sample, share of a tile's columns) ----------------
    // Per 32 columns the bias is added; then, threshold pass: the scores are written out; filter pass: which of them
    // reach the sample's threshold (32 independent comparisons, a bit each), then the appends of those that do.
    const int q = warp & 3;                 // a warp reaches the 32 lanes of tensor memory of its number modulo four
    const int half = (warp - 3) >> 2;       // which share of a tile's 128 columns
    const int row = 32 * q + lane;          // sample inside the block
    const int et = tid - 96;                // the first 128 read-back threads fetch the tile's biases
    const int vslice = slice * TC_SPLIT + half;    // buffers are kept per (slice, share of the columns)
    int2* mybuf = p.cand + ((size_t)vslice * p.Bpad + s0 + row) * p.gbuf;
    const float tau = DUMP ? 0.f : p.tau[s0 + row];
    int cnt = 0;
    if (DUMP && slice == 0 && half == 0) {      // the threshold pass also clears what the filter pass accumulates into
      if (s0 + row < p.B) p.need_fix[s0 + row] = 0;
      if (tid == 96 && blockIdx.y == 0) *p.norm2max = 0u;
    }
    if (half == 0) {
      // the block's activations -> tensor memory: lane = sample, column = hidden unit (samples past the batch: zeros)
      const float4* hrow = reinterpret_cast<const float4*>(p.h + (size_t)(s0 + row) * p.H);
      const bool live = s0 + row < p.B;
      for (int c0 = 0; c0 < p.H; c0 += 32) {
        uint32_t r[32];
#pragma unroll
        for (int c4 = 0; c4 < 8; ++c4) {
          const float4 v = live ? __ldg(hrow + (c0 >> 2) + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
          r[4 * c4] = __float_as_uint(v.x); r[4 * c4 + 1] = __float_as_uint(v.y);
          r[4 * c4 + 2] = __float_as_uint(v.z); r[4 * c4 + 3] = __float_as_uint(v.w);
        }
        tc_st32(tmem_base + ((uint32_t)(32 * q) << 16) + acol + (uint32_t)c0, r);
      }
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      tc_bar_arrive(bar_a);
    }
    // a tile's biases are asked for one tile ahead, so that their latency is not part of the tile's read-back
    auto bias_of = [&](int i) {
      const int j = (slice + i * p.nslices) * p.tile_stride * TC_N + et;
      return et < TC_N && i < my_tiles && j < p.N ? __ldg(&p.hdr2[j].b) : 0.f;
    };
    float bias_next = bias_of(0);
    int acc = 0, accround = 0;
    for (int i = 0; i < my_tiles; ++i) {
      const int tile = slice + i * p.nslices;
      const int j0 = tile * p.tile_stride * TC_N;
      if (et < TC_N) sb[acc * TC_N + et] = bias_next;
      bias_next = bias_of(i + 1);
      if (warp == 3) tc_bar_wait(bar_accfull + acc, accround & 1, abort_flag);      // one warp polls, the others sleep in the barrier
      asm volatile("bar.sync 1, %0;" ::"n"(TC_EPI) : "memory");          // the accumulator is complete, the tile's biases are in place
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      for (int c0 = (TC_N / TC_SPLIT) * half; c0 < (TC_N / TC_SPLIT) * (half + 1); c0 += 32) {
        uint32_t r[32];
        tc_ld32(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(acc * TC_N + c0), r);
        const int jb = j0 + c0;
        const float4* sb4 = reinterpret_cast<const float4*>(sb + acc * TC_N + c0);
        unsigned hm = 0u;
#pragma unroll
        for (int c4 = 0; c4 < 8; ++c4) {
          const float4 bq = sb4[c4];
          const float z0 = __uint_as_float(r[4 * c4]) + bq.x, z1 = __uint_as_float(r[4 * c4 + 1]) + bq.y;
          const float z2 = __uint_as_float(r[4 * c4 + 2]) + bq.z, z3 = __uint_as_float(r[4 * c4 + 3]) + bq.w;
          r[4 * c4] = __float_as_uint(z0); r[4 * c4 + 1] = __float_as_uint(z1);
          r[4 * c4 + 2] = __float_as_uint(z2); r[4 * c4 + 3] = __float_as_uint(z3);
          if (!DUMP) {
            if (z0 >= tau) hm |= 1u << (4 * c4);
            if (z1 >= tau) hm |= 2u << (4 * c4);
            if (z2 >= tau) hm |= 4u << (4 * c4);
            if (z3 >= tau) hm |= 8u << (4 * c4);
          }
        }
        if (DUMP) {
          // neurons past the end score -infinity; a thread's 32 scores are 128 contiguous bytes
          float4* out = reinterpret_cast<float4*>(p.dump + (size_t)(s0 + row) * p.dump_cols + (size_t)tile * TC_N + c0);
#pragma unroll
          for (int c4 = 0; c4 < 8; ++c4) {
            float4 v;
            v.x = jb + 4 * c4 < p.N ? __uint_as_float(r[4 * c4]) : -INFINITY;
            v.y = jb + 4 * c4 + 1 < p.N ? __uint_as_float(r[4 * c4 + 1]) : -INFINITY;
            v.z = jb + 4 * c4 + 2 < p.N ? __uint_as_float(r[4 * c4 + 2]) : -INFINITY;
            v.w = jb + 4 * c4 + 3 < p.N ? __uint_as_float(r[4 * c4 + 3]) : -INFINITY;
            __stcg(out + c4, v);
          }
        } else {
          if (p.N - jb < 32) hm &= p.N > jb ? (1u << (p.N - jb)) - 1u : 0u;      // neurons past the end (last tile only)
          // the columns that some sample of the warp keeps (few): one more read of that column, same sum as above
          unsigned any = __reduce_or_sync(0xffffffffu, hm);
          while (any) {
            const int c = __ffs(any) - 1;
            any &= any - 1;
            uint32_t raw;
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];\n\ttcgen05.wait::ld.sync.aligned;"
                         : "=r"(raw) : "r"(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(acc * TC_N + c0 + c)) : "memory");
            if ((hm >> c) & 1u) {
              const float z = __uint_as_float(raw) + sb[acc * TC_N + c0 + c];
              if (cnt < p.gbuf) __stcg(mybuf + cnt, make_int2(__float_as_int(z), jb + c));
              ++cnt;
            }
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      tc_bar_arrive(bar_accempty + acc);
      if (++acc == nacc) { acc = 0; ++accround; }
    }
    if (!DUMP && s0 + row < p.B) {
      p.cand_cnt[(size_t)vslice * p.Bpad + s0 + row] = cnt < p.gbuf ? cnt : p.gbuf;
      if (cnt > p.gbuf) p.need_fix[s0 + row] = 1;          // candidates were dropped: the sample is scored exactly
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TC_TMEM_COLS) : "memory");
  }
  if (tid == 0 && *abort_flag) atomicCAS(&p.st->status, 0, (int)DSLIDE_ERR_TIMEOUT);
}

// Floats as keys that order like them (unsigned); no real score has key 0.
__device__ __forceinline__ uint32_t tc_key(float z) {
  const uint32_t b = __float_as_uint(z);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float tc_unkey(uint32_t k) { return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k); }
// The cap-th largest of the block's per-thread keys, found bit by bit (a block-wide count per bit); 0 when fewer than
// cap threads hold a key.
__device__ __forceinline__ uint32_t tc_select(uint32_t mine, int cap) {
  uint32_t K = 0u;
  for (int bit = 31; bit >= 0; --bit) {
    const uint32_t trial = K | (1u << bit);
    if (__syncthreads_count(mine >= trial) >= cap) K = trial;
  }
  return K;
}

// One block per sample.  Each thread takes the largest of its share of the sample's scores of the subset; the cap-th
// largest of these maxima is the sample's threshold.  At least cap neurons of the subset reach it (exactly cap when
// the cap best fell to different threads); -infinity when the subset is smaller than that.  Any threshold gives the
// same results: it only decides how many candidates the filter pass hands on.
constexpr int TAU_THREADS = 256;
__global__ void __launch_bounds__(TAU_THREADS) k_tc_tau(const float* dump, int cols, int rank, float* tau) {
  const int s = blockIdx.x, tid = threadIdx.x;
  griddep_launch_dependents();
  griddep_wait();                    // the threshold pass has completed
  uint32_t mine = 0u;
  for (int e = tid; e < cols; e += TAU_THREADS) {
    const uint32_t key = tc_key(__ldcg(dump + (size_t)s * cols + e));
    mine = key > mine ? key : mine;
  }
  const uint32_t K = tc_select(mine, rank);
  if (tid == 0) {
    float t = tc_unkey(K);
    if (K == 0u || !(t == t)) t = -INFINITY;      // everything passes
    tau[s] = t;
  }
}

// A flagged sample: every neuron scored exactly in fp32 by the sample's block (rare; the block walks all of W2).
// fx_smem: [H] activation, then [warps][k] lists of scores and of ids, then the lists' lengths.
constexpr int FX_THREADS = 256;
__device__ void tc_exact_scan(float* fx_smem, int s, const float* W2, const RowHdr* hdr2, const float* h, int H, int N, int k,
                              int32_t* out_ids, float* out_scores) {
  float* hs = fx_smem;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = FX_THREADS / 32;
  float* wz = hs + H + warp * k;
  int* wi = reinterpret_cast<int*>(hs + H + nw * k) + warp * k;
  for (int c = tid; c < H; c += FX_THREADS) hs[c] = h[(size_t)s * H + c];
  __syncthreads();
  const int H4 = H >> 2;
  const float4* h4 = reinterpret_cast<const float4*>(hs);
  int cnt = 0;                                  // lane 0: entries of the warp's list
  for (int j = warp; j < N; j += nw) {
    const float4* r = reinterpret_cast<const float4*>(W2 + (size_t)j * H);
    float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;
    for (int c = lane; c < H4; c += 32) {
      const float4 w = __ldg(r + c), x = h4[c];
      d0 = fmaf(w.x, x.x, d0); d1 = fmaf(w.y, x.y, d1); d2 = fmaf(w.z, x.z, d2); d3 = fmaf(w.w, x.w, d3);
    }
    float d = (d0 + d1) + (d2 + d3);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
    if (lane == 0) {
      const float z = __ldg(&hdr2[j].b) + d;
      if (cnt < k || tc_better(z, j, wz[cnt - 1], wi[cnt - 1])) {
        int at = cnt < k ? cnt++ : k - 1;
        while (at > 0 && tc_better(z, j, wz[at - 1], wi[at - 1])) { wz[at] = wz[at - 1]; wi[at] = wi[at - 1]; --at; }
        wz[at] = z; wi[at] = j;
      }
    }
  }
  int* cnts = reinterpret_cast<int*>(hs + H + 2 * nw * k);
  if (lane == 0) cnts[warp] = cnt;
  __syncthreads();
  if (tid == 0) {
    int head[FX_THREADS / 32];
    for (int w = 0; w < nw; ++w) head[w] = 0;
    float* az = hs + H;
    int* ai = reinterpret_cast<int*>(hs + H + nw * k);
    for (int qk = 0; qk < k; ++qk) {
      int bw = -1;
      for (int w = 0; w < nw; ++w) {
        if (head[w] >= cnts[w]) continue;
        if (bw < 0 || tc_better(az[w * k + head[w]], ai[w * k + head[w]], az[bw * k + head[bw]], ai[bw * k + head[bw]])) bw = w;
      }
      out_ids[(size_t)s * k + qk] = bw >= 0 ? ai[bw * k + head[bw]] : -1;
      out_scores[(size_t)s * k + qk] = bw >= 0 ? az[bw * k + head[bw]] : -INFINITY;
      if (bw >= 0) head[bw]++;
    }
  }
}

// One block per sample: the slices' candidates -> those whose approximate score reaches the cap-th largest of the
// threads' maxima (cap of them, or a few more) -> their exact fp32 logits -> the k best by (logit descending, id
// ascending).  need_fix[s] = 1 when the filter cannot be shown to be exact.
constexpr int RF_THREADS = FX_THREADS;
constexpr int RF_MAXV = 512;       // buffers per sample at most
constexpr int RF_SLOTS = 64;       // candidates scored exactly at most
__global__ void __launch_bounds__(RF_THREADS)
k_tc_refine(const float* W2, const RowHdr* hdr2, const float* h, const int2* cand, const int* cand_cnt, int gbuf, const float* tau, int Bpad,
            const unsigned int* norm2max, int B, int H, int N, int cap, int nvs, int k, int32_t* out_ids, float* out_scores,
            const int* need_fix) {
  __shared__ float fx_space[1024];               // the exact scan's work space (H <= 256 activations + 2 x 8 x 8 list entries + 8)
  __shared__ int offs[RF_MAXV + 1];
  __shared__ float ez[RF_SLOTS], sz[RF_SLOTS];
  __shared__ int ei[RF_SLOTS], si[RF_SLOTS];
  __shared__ float red[RF_THREADS / 32];
  __shared__ int wsum[RF_THREADS / 32];
  __shared__ int sh_n, sh_fix;
  const int s = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  griddep_wait();                                // the filter pass has completed
  // fill of the sample's buffers -> their places in one list (exclusive scan; each thread owns RF_MAXV / RF_THREADS buffers)
  {
    constexpr int PER = RF_MAXV / RF_THREADS;
    int c[PER], mine = 0;
#pragma unroll
    for (int i = 0; i < PER; ++i) { const int v = tid * PER + i; c[i] = v < nvs ? __ldcg(cand_cnt + (size_t)v * Bpad + s) : 0; mine += c[i]; }
    int inc = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const int o = __shfl_up_sync(0xffffffffu, inc, d); if (lane >= d) inc += o; }
    if (lane == 31) wsum[warp] = inc;
    if (tid == 0) { sh_n = 0; sh_fix = need_fix[s]; }      // a buffer of the sample ran over in the filter pass
    __syncthreads();
    int base = 0;
    for (int w = 0; w < warp; ++w) base += wsum[w];
    int run = base + inc - mine;
#pragma unroll
    for (int i = 0; i < PER; ++i) { offs[tid * PER + i] = run; run += c[i]; }
    if (tid == RF_THREADS - 1) offs[RF_MAXV] = run;
    __syncthreads();
  }
  const int total = offs[RF_MAXV];
  int nc = 0;
  uint32_t K = 0u;
  bool fix = false;
  {
  // Entry e of the sample's list lies in the buffer v with offs[v] <= e < offs[v + 1].  First walk: a thread keeps the
  // largest key of its entries.  The candidates that reach the cap-th largest of these maxima go on (all of them when
  // there are no more than cap): a second walk over the same entries (they are in L2) collects them.
  auto entry = [&](int e) {
    int lo = 0, hi = RF_MAXV;                     // invariant: offs[lo] <= e < offs[hi]
    while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (offs[mid] <= e) lo = mid; else hi = mid; }
    return __ldcg(cand + ((size_t)lo * Bpad + s) * gbuf + (e - offs[lo]));
  };
  constexpr int KEEP = 8;                         // entries per thread that stay in registers between the walks
  int2 keep[KEEP];
  uint32_t mine = 0u;
#pragma unroll
  for (int i = 0; i < KEEP; ++i) {
    const int e = tid + i * RF_THREADS;
    keep[i] = e < total ? entry(e) : make_int2(0, 0);
    const uint32_t key = e < total ? tc_key(__int_as_float(keep[i].x)) : 0u;
    mine = key > mine ? key : mine;
  }
  for (int e = tid + KEEP * RF_THREADS; e < total; e += RF_THREADS) {
    const uint32_t key = tc_key(__int_as_float(entry(e).x));
    mine = key > mine ? key : mine;
  }
  K = total > cap ? tc_select(mine, cap) : 0u;
#pragma unroll
  for (int i = 0; i < KEEP; ++i)
    if (tid + i * RF_THREADS < total && tc_key(__int_as_float(keep[i].x)) >= K) {
      const int slot = atomicAdd(&sh_n, 1);
      if (slot < RF_SLOTS) ei[slot] = keep[i].y;
    }
  for (int e = tid + KEEP * RF_THREADS; e < total; e += RF_THREADS) {
    const int2 x = entry(e);
    if (tc_key(__int_as_float(x.x)) >= K) { const int slot = atomicAdd(&sh_n, 1); if (slot < RF_SLOTS) ei[slot] = x.y; }
  }
  __syncthreads();
  nc = sh_n;
  fix = nc > RF_SLOTS;                            // many equal scores at the cut: the sample is scored exactly
  }
  if (!fix) {
  // exact logits of the kept candidates: a warp per candidate, four partial sums per lane as in the exact path
  const float4* h4 = reinterpret_cast<const float4*>(h + (size_t)s * H);
  const int H4 = H >> 2;
  for (int e = warp; e < nc; e += RF_THREADS / 32) {
    const int j = ei[e];
    const float4* r = reinterpret_cast<const float4*>(W2 + (size_t)j * H);
    float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;
    for (int c = lane; c < H4; c += 32) {
      const float4 w = __ldg(r + c), x = h4[c];
      d0 = fmaf(w.x, x.x, d0); d1 = fmaf(w.y, x.y, d1); d2 = fmaf(w.z, x.z, d2); d3 = fmaf(w.w, x.w, d3);
    }
    float d = (d0 + d1) + (d2 + d3);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
    if (lane == 0) ez[e] = __ldg(&hdr2[j].b) + d;
  }
  // |h|^2 of the sample
  float hs = 0.f;
  for (int c = tid; c < H; c += RF_THREADS) { const float x = h[(size_t)s * H + c]; hs += x * x; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) hs += __shfl_xor_sync(0xffffffffu, hs, o);
  if (lane == 0) red[warp] = hs;
  __syncthreads();
  // order the exact scores: an entry's place is the number of better ones ((score, id) pairs are all different)
  if (tid < nc) {
    const float z = ez[tid]; const int j = ei[tid];
    int rank = 0;
    for (int u = 0; u < nc; ++u) rank += tc_better(ez[u], ei[u], z, j) ? 1 : 0;
    sz[rank] = z; si[rank] = j;
  }
  __syncthreads();
  if (tid < k) {
    out_ids[(size_t)s * k + tid] = tid < nc ? si[tid] : -1;
    out_scores[(size_t)s * k + tid] = tid < nc ? sz[tid] : -INFINITY;
  }
  if (tid == 0) {
    float hn = 0.f;
    for (int w = 0; w < RF_THREADS / 32; ++w) hn += red[w];
    // Every neuron that did not go on to the exact pass has an approximate score below T: the cut when candidates
    // were dropped here, else the sample's threshold (a neuron below it was never a candidate).  Its exact score is
    // at most T plus the error bound; the k best are certain when the k-th exact score lies above.
    const float T = total > cap ? tc_unkey(K) : tau[s];
    if (T > -INFINITY) {
      const float bound = T + TC_ERR * sqrtf(hn) * sqrtf(__uint_as_float(*norm2max)) + 1e-30f;
      const int kth = (k < nc ? k : nc) - 1;
      if (nc < k || !(sz[kth] > bound)) sh_fix = 1;
    }
  }
  }
  __syncthreads();
  if (fix || sh_fix) tc_exact_scan(fx_space, s, W2, hdr2, h, H, N, k, out_ids, out_scores);
}

// ---------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// rows x H fp32, row-major; boxes of 128 rows x 32 units, 128-byte swizzle; rows past the end read as zero
static bool make_map(CUtensorMap* m, const float* base, int rows, int H) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)H, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)H * 4};
  const cuuint32_t box[2] = {(cuuint32_t)TC_KB, (cuuint32_t)TC_M};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool dense_tc_usable(const Ctx* c, int k) {
  return k >= 1 && k <= TC_K_MAX && c->H % TC_KB == 0 && c->H >= TC_KB && c->H <= 256 && c->N >= TC_N && encode_fn() != nullptr;
}

// The hidden activations of the batch are in c->h (left there by the forward kernel in predict mode).
cudaError_t launch_dense_tc(Ctx* c, int batch, int k, int32_t* out_ids, float* out_scores) {
  const int cap = 2 * k + TC_EXTRA;
  const int groups = (batch + TC_M - 1) / TC_M;
  const int ntiles = (c->N + TC_N - 1) / TC_N;
  int nslices = c->num_sms / groups;
  if (nslices < 1) nslices = 1;
  if (nslices > ntiles) nslices = ntiles;
  if (TC_SPLIT * nslices > RF_MAXV) nslices = RF_MAXV / TC_SPLIT;      // k_tc_refine's table of buffer offsets
  // threshold pass: every `stride`-th tile, at most TAU_MAX_TILES of them
  constexpr int TAU_MAX_TILES = 128;
  int stride = TC_SUBSET;
  if ((ntiles + stride - 1) / stride > TAU_MAX_TILES) stride = (ntiles + TAU_MAX_TILES - 1) / TAU_MAX_TILES;
  const int nsub = (ntiles + stride - 1) / stride;
  const int dump_cols = nsub * TC_N;
  int nslices_sub = nslices < nsub ? nslices : nsub;
  // work space: the norm bound, the flags, the thresholds, the candidate buffers of every slice and their fill, the
  // threshold pass's scores
  const int Bpad = groups * TC_M;
  const int nvs = TC_SPLIT * nslices;
  auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
  const size_t off_fix = 256, off_tau = off_fix + up((size_t)Bpad * 4), off_cnt = off_tau + up((size_t)Bpad * 4);
  const size_t off_cand = off_cnt + up((size_t)nvs * Bpad * 4);
  // The threshold is the rank-th best of the subset's maxima, the rank chosen so that about TC_TARGET x cap neurons
  // reach it over all N whatever the subset's share; a buffer has room for four times its expected fill.
  int rank = (cap * TC_TARGET + stride - 1) / stride;
  if (rank > cap) rank = cap;
  if (rank < 4) rank = 4;
  int gbuf = TC_GBUF_MIN;
  while (gbuf * nvs < 4 * rank * stride) gbuf <<= 1;
  const size_t off_dump = off_cand + up((size_t)nvs * Bpad * gbuf * sizeof(int2));
  const size_t need = off_dump + (size_t)Bpad * dump_cols * 4;
  cudaError_t e;
  if (need > c->pd_cap) {
    if ((e = cudaStreamSynchronize(c->stream)) != cudaSuccess) return e;
    if (c->pd_part) cudaFree(c->pd_part);
    c->pd_part = nullptr; c->pd_cap = 0;
    if ((e = cudaMalloc(&c->pd_part, need)) != cudaSuccess) return e;
    c->pd_cap = need;
  }
  unsigned char* ws = reinterpret_cast<unsigned char*>(c->pd_part);
  unsigned int* norm2 = reinterpret_cast<unsigned int*>(ws);
  int* need_fix = reinterpret_cast<int*>(ws + off_fix);
  float* tau = reinterpret_cast<float*>(ws + off_tau);
  int* cand_cnt = reinterpret_cast<int*>(ws + off_cnt);
  int2* cand = reinterpret_cast<int2*>(ws + off_cand);
  float* dump = reinterpret_cast<float*>(ws + off_dump);

  CUtensorMap tmW;
  if (!make_map(&tmW, c->W2, c->N, c->H)) return cudaErrorInvalidValue;


  TcParams p;
  p.hdr2 = c->hdr2; p.h = c->h; p.cand = cand; p.cand_cnt = cand_cnt; p.dump = dump; p.tau = tau; p.need_fix = need_fix; p.norm2max = norm2; p.st = c->dstate;
  p.B = batch; p.Bpad = Bpad; p.H = c->H; p.N = c->N; p.dump_cols = dump_cols; p.gbuf = gbuf;
  const size_t tile_bytes = (size_t)(c->H / TC_KB) * TC_SUB_BYTES;
  int stages = (int)(((size_t)200 << 10) / tile_bytes);
  if (stages > TC_STAGES) stages = TC_STAGES;
  p.stages = stages;
  const size_t smem = 1024 + tile_bytes * stages + TC_NACC * TC_N * 4 + 24 * 8 + 64;
  if ((e = cudaFuncSetAttribute(k_dense_tc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(k_dense_tc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
  {
    LaunchScope ls(c, KID_PREDICT);
    p.nslices = nslices_sub; p.ntiles = nsub; p.tile_stride = stride;
    // each kernel of the call may be placed while the kernel before it drains (they wait for it before they read or
    // write anything); the first follows the hidden-layer kernel in the same way
    if ((e = launch_dependent(k_dense_tc<true>, dim3(nslices_sub, groups), dim3(TC_THREADS), smem, c->stream, tmW, p)) != cudaSuccess) return e;
    if ((e = launch_dependent(k_tc_tau, dim3(Bpad), dim3(TAU_THREADS), 0, c->stream, (const float*)dump, dump_cols, rank, tau)) != cudaSuccess)
      return e;
    p.nslices = nslices; p.ntiles = ntiles; p.tile_stride = 1;
    if ((e = launch_dependent(k_dense_tc<false>, dim3(nslices, groups), dim3(TC_THREADS), smem, c->stream, tmW, p)) != cudaSuccess) return e;
    if ((e = launch_dependent(k_tc_refine, dim3(batch), dim3(RF_THREADS), 0, c->stream, (const float*)c->W2, (const RowHdr*)c->hdr2,
                              (const float*)c->h, (const int2*)cand, (const int*)cand_cnt, gbuf, (const float*)tau, Bpad,
                              (const unsigned int*)norm2, batch, c->H, c->N, cap, nvs, k, out_ids, out_scores, (const int*)need_fix)) !=
        cudaSuccess)
      return e;
  }
  return cudaGetLastError();
}

}  // namespace dslide
