// Internal declarations of libdslide (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/dslide.h"

namespace dslide {

// ---------------------------------------------------------------------------
// Counter-based random numbers: three rounds of the splitmix64 output function
// over (seed, stream, rebuild count, counter).  Used for the initial weights and
// for the hash functions of every rebuild (Algorithm 1: "Rebuild hash tables and
// hash functions").
// ---------------------------------------------------------------------------
__host__ __device__ inline uint64_t sm64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
__host__ __device__ inline uint64_t ctr_rng(uint64_t seed, uint64_t stream, uint64_t r, uint64_t ctr) {
  const uint64_t g = 0x9E3779B97F4A7C15ull;
  uint64_t a = sm64(seed + g * (stream + 1));
  uint64_t b = sm64(a + g * (r + 1));
  return sm64(b + g * (ctr + 1));
}
enum : uint64_t { RNG_W1 = 0, RNG_W2 = 1, RNG_HASH = 2, RNG_PROBE = 3, RNG_SAMPLE = 4, RNG_FILL = 5, RNG_HASH1 = 6 };
constexpr int DENSIFY_ATTEMPTS = 16;     // functions an all-zero DWTA bin of a query probes for a position to borrow

// Device-resident step state (read and written by kernels only; the host reads it
// in the synchronous statistics and status calls).
struct DevState {
  int status;                      // sticky dslide_status seen on the device
  int pad0[3];
  // Slots indexed by the parity of the step: the kernels of step t use slot t & 1 and the update
  // kernel zeroes the other slot for step t + 1.
  unsigned int n_own[2][2];        // distinct touched rows of W2 ([.][0]) and W1 ([.][1]): lengths of the row lists
  unsigned int n_hot[2];           // rows touched by more than HOT_T samples (entries of the hot-row list)
  unsigned int n_med[2];           // rows touched by more than ROW_SLOTS samples (entries of the medium-row list)
  unsigned int ticket[2];          // work tickets handed out by the update kernel
  unsigned int n_hotslots;         // rows of W1 that were given a line of the coefficient table so far (not per step)
  unsigned long long acc[2][3];    // forward kernel: sum of active-set sizes, nonzeros, bucket entries read
  unsigned long long last[3];      // acc of the last finished step
  unsigned long long cum[6];       // since the last reset: steps, sum_active, U2, U1, nnz, fetched
};

// What a host-buffer step reports straight into pinned host memory: the update kernel writes status and loss,
// then (after a system-wide fence) the step's sequence number, which the host polls.
constexpr int ST_SETS = 3;      // staging sets of the host-buffer steps
struct HostResult {
  unsigned int seq;
  int status;
  float loss;
  int pad;
};

// Touches of a row of W1 / W2 whose (sample, coefficient) pair is stored with the row; further touches of the
// same step only set the sample's bit in the row's mask.
constexpr int ROW_SLOTS = 6;
// A row touched by more than HOT_T samples of a step is listed by the forward kernel (top bit of its
// count set) and summed in HOT_SLICES slices by different warps; at most HOT_CAP rows are listed, further
// ones are summed by a single warp.
constexpr int HOT_T = 32;
// Touches of a row up to this many keep their (sample, coefficient) pair (the first ROW_SLOTS in the row record).
constexpr int PAIR_T = 32;
// Rows of W1 that have been hot once (frequent features stay frequent) own a line of a coefficient table: every
// later touch leaves its value there, indexed by sample, and the slices of the row read it instead of searching.
constexpr int HOTMAP_CAP = 4096;
constexpr int HOT_SLICES = 8;
constexpr int HOT_CAP = 1024;
// Rows touched by more than ROW_SLOTS samples are listed too (at most MED_CAP of them; further ones are found
// by the warp that walks the ordinary row list).  A row's count word: low bits = touching samples, CNT_MED /
// CNT_HOT = the row is on the medium / hot list.
constexpr int MED_CAP = 65536;
constexpr unsigned CNT_HOT = 0x80000000u, CNT_MED = 0x40000000u, CNT_MASK = 0x3fffffffu;

// Per-row record next to a row of W1 / W2, one 64-byte line: the number of samples of the step in flight that
// touch the row (plus the CNT_* list marks), the row's bias with its Adam moments (rows of W2 only) and the
// (sample, coefficient bits) pairs of the row's first ROW_SLOTS touches.  The update kernel fetches it together
// with the row.
struct __align__(16) RowHdr {
  uint32_t cnt;
  float b, mb, vb;
  int2 slot[ROW_SLOTS];
};
static_assert(sizeof(RowHdr) == 64, "the row record is one 64-byte line");

// Programmatic dependent launch: a kernel launched with launch_dependent() may become resident while the kernel
// before it in the stream is still running; it must not touch anything that kernel reads or writes before
// griddep_wait(), which returns once that kernel has completed and its writes are visible.
// griddep_launch_dependents() tells the runtime that the next kernel may start to be placed.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                    Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

struct Ctx;

// Kernel ids for the per-kernel timing (must match the DSLIDE_K_* enum of the C ABI).
enum { KID_FORWARD = 0, KID_ADAM_DENSE, KID_ADAM, KID_DRAW_HASH, KID_HASH_NEURONS, KID_BUCKET_SCAN, KID_SORT_HIST,
       KID_SORT_SCAN, KID_SORT_SCATTER, KID_PREDICT, KID_INIT, KID_PLACE_IDS, KID_ORDER_BUCKETS, KID_COUNT };

// Brackets one kernel launch: counts it and, while profiling is on, records a CUDA event pair around it.
struct LaunchScope {
  Ctx* c; int kid; long long rec;      // rec: index of the event pair in the context's list, -1 when not profiling
  LaunchScope(Ctx* c, int kid);
  ~LaunchScope();
};

// launches (implemented in the .cu files)
cudaError_t launch_init_gauss(Ctx* c, float* w, int64_t n, uint64_t stream_id);
cudaError_t launch_draw_hash(Ctx* c, int64_t r);
cudaError_t launch_build_tables(Ctx* c);
cudaError_t launch_draw_proj1(Ctx* c, int64_t r);   // the hidden layer's projections of rebuild count r
cudaError_t launch_build_tables1(Ctx* c);           // codes of the hidden neurons and their tables
cudaError_t launch_order_buckets(Ctx* c, int min_n);
cudaError_t launch_forward_train(Ctx* c, int batch, const int32_t* row_ptr, const int32_t* col_idx,
                                 const float* vals, const int32_t* label_ptr, const int32_t* labels, int inputs_ready);
cudaError_t launch_update(Ctx* c, int batch, const int32_t* row_ptr, const int32_t* col_idx, const float* vals,
                          float* loss_out, HostResult* host_res, unsigned int host_seq);
cudaError_t launch_predict(Ctx* c, int batch, const int32_t* row_ptr, const int32_t* col_idx,
                           const float* vals, int k, int dense, int32_t* out_ids, float* out_scores);
bool dense_tc_usable(const Ctx* c, int k);           // inference over all neurons on the tensor pipe: shapes it covers
cudaError_t launch_dense_tc(Ctx* c, int batch, int k, int32_t* out_ids, float* out_scores);
cudaError_t setup_forward(Ctx* c);   // chooses the dedup path and the shared-memory layout

struct Ctx {
  dslide_config cfg;
  int D, H, N, K, L, KL;
  int bits;            // bits of a bucket code
  int lg_bin;          // log2(dwta bin)
  int fn_len;          // indices per hash function: srp_nnz (SimHash) or bin (DWTA)
  int cap;
  int64_t nb;          // buckets per table = 2^bits
  int act_stride;      // row stride of the per-sample active arrays
  int Wd;              // 32-bit words of a per-row sample mask = ceil(max_batch / 32)
  int dense;
  cudaStream_t stream;

  float *W1, *b1, *W2;
  float *mW1, *vW1, *mb1, *vb1, *mW2, *vW2;
  RowHdr *hdr1, *hdr2;             // per row of W1 / W2: touch count, slots and (W2) the bias b2 with its moments
  int32_t *hash_idx, *hash_sign;
  int32_t *bucket_off, *bucket_ids;
  // LSH-sampled hidden layer (hidden_L > 0): projections over the input coordinates, tables over the hidden neurons,
  // per-step codes and active masks, per row of W1 the hidden units some sample of the step touches it for
  int K1, L1, KL1, cap1, Hw;       // Hw = 32-bit words of a mask over the hidden units
  int8_t* proj1;                   // [D][KL1]
  int32_t *bucket1_off, *bucket1_ids;
  uint32_t *codes1n;               // [L1][H] codes of the hidden neurons (table build)
  uint32_t *codes1, *hmask;        // [B][L1], [B][Hw]
  uint32_t* cmask1;                // [D][Hw]

  // per-step work space
  float *h, *dh, *loss;
  uint32_t* codes;
  int32_t *act_cnt, *act_ids;
  float *act_z, *act_p, *act_g;
  uint32_t *mask1, *mask2;         // per row of W1 / W2: which samples of the batch touch it
  int32_t* hotmap1;                // per row of W1: its line of hotcoef1, or -1
  float* hotcoef1;                 // [HOTMAP_CAP][max_batch]
  int2 *ovf1, *ovf2;               // per row: the (sample, coefficient) pairs of touches ROW_SLOTS .. PAIR_T - 1, at [row][touch]
  int2 *own1, *own2;               // the distinct touched rows of W1 / W2 with their first-touching sample, in no particular order
  int32_t* hot_rows;               // rows touched by many samples: row of W2, or ~row of W1
  int32_t* med_rows;               // rows touched by more than ROW_SLOTS samples, same encoding
  float* hot_part;                 // [HOT_CAP][HOT_SLICES][H + 4] slice sums of those rows
  int* hot_done;                   // [HOT_CAP] finished slices per listed row (returns to 0)
  DevState* dstate;

  // rebuild work space
  uint32_t *keysA, *keysB;
  int32_t *valsA, *valsB;
  int32_t* tile_hist;
  int32_t* bucket_part;   // per table: sums of chunks of bucket counters (bucket offset scan)
  int place_path;         // 1: codes wider than a radix digit: ids placed by atomics, then ordered inside buckets
  int2 *ord_mid, *ord_big; // (table, bucket) of the buckets too large to order in registers / in shared memory
  int* ord_cnt;           // lengths of those two lists
  int ids_ordered_above;  // place path: buckets with more ids than this are in ascending order (1 = every bucket)
  int sort_passes, sort_width, sort_tiles;

  // forward kernel layout
  int dedup_mode;      // 1 bitmap, 2 sort
  int fwd_smem;        // dynamic shared memory of the forward kernel
  int fwd_stage_bytes; // of which: staging space for rows of W1 / W2 (overlays the dedup work space)
  int fwd_hash_sm_off, fwd_hash_sm_bytes;  // the hash functions' mirror inside the forward kernel's staging region (-1: none)
  int fwd_sort_small;  // candidate sets up to this size are deduplicated by sorting
  int sort_cap;        // capacity (power of two) of the shared-memory sort buffer
  int num_sms;

  // staging for the host-buffer entry point
  // host-buffer entry points: two sets of (device buffer, pinned host buffer, pinned result, event), used in turn
  // Three sets in rotation: when step t is packed, the result of step t - 2 has been collected, which proves
  // that every kernel up to the forward kernel of step t - 2 has finished -- so the set of step t - 3 is free,
  // while the update kernel of step t - 2 may still be reading its own.
  unsigned char *st_dev[ST_SETS], *st_host[ST_SETS];
  int64_t st_cap[ST_SETS];
  HostResult *st_res[ST_SETS], *st_res_dev[ST_SETS];   // pinned, device-mapped: what the update kernel reports of the step that used the set
  unsigned int st_seq[ST_SETS];                  // sequence number that step was given
  unsigned int st_counter;                 // sequence numbers handed out so far
  cudaEvent_t st_in[ST_SETS];                    // input copy finished
  cudaStream_t st_copy_in;                 // the input copy runs beside the kernels of the previous step
  int st_pending[ST_SETS];          // a step was enqueued on the set and its result has not been handed out yet
  int st_next;                // set the next host-buffer step uses

  int64_t t_host, r_host, next_rebuild;
  int64_t launches;
  int profiling;
  void* pd_part;       // dense inference: the slices' best-k lists (ids, then scores), grown on demand
  size_t pd_cap;
  void* prof;          // std::vector of event pairs while profiling
};

}  // namespace dslide
