/*
 * dslide.h -- C ABI of libdslide: the SLIDE adaptive-sparse training step of a
 * two-layer fully connected network (sparse input -> dense ReLU hidden layer ->
 * LSH-sampled softmax output layer) on one NVIDIA B200 (sm_100a).
 *
 * The operations follow "Distributed SLIDE" (arXiv 2201.12667): Section 2.1 (the
 * three phases of SLIDE), Algorithm 1 (training procedure), Section 3.5 (Adam
 * moments per weight and bias array), Section 3.6 (layer operations and the
 * per-sample snapshot of active neurons), Section 3.7 (sampling budget), Section 4.1
 * (hash families, K, L, Adam constants).  Nothing is sharded or communicated between GPUs.
 *
 * Conventions
 *  - Every function returns a dslide_status.  No exceptions, no abort, no output.
 *  - "device" pointers are CUDA device pointers on the context's device, owned by
 *    the caller, read-only unless stated, and must stay valid until the work
 *    enqueued by the call has finished on the context's stream.
 *  - Calls are asynchronous on the context's stream unless stated.  Errors the
 *    host can see (bad arguments, wrong state) are returned at once and the call
 *    has no effect.  Errors only the device can see (feature or label id out of
 *    range, active set larger than configured) set a sticky status word; the
 *    offending sample is skipped (it contributes no loss and no gradient), no
 *    out-of-bounds access is made, and the status is returned, and cleared, by
 *    the next dslide_sync.
 *  - The context owns the model state, the hash tables and all work space.
 *    One context must not be used from two host threads at once.
 *  - Matrices are row-major fp32: W1[D][H], W2[N][H]; ids are int32.
 */
#ifndef DSLIDE_H
#define DSLIDE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dslide_ctx dslide_ctx;

typedef enum {
  DSLIDE_OK = 0,
  DSLIDE_ERR_INVALID_ARG = 1,
  DSLIDE_ERR_OOM = 2,
  DSLIDE_ERR_CUDA = 3,
  DSLIDE_ERR_OVERFLOW = 4,   /* an active set, label list or batch exceeds the configured maximum */
  DSLIDE_ERR_BAD_INDEX = 5,  /* feature id outside [0,D) or label id outside [0,N), seen on the device */
  DSLIDE_ERR_STATE = 6,
  DSLIDE_ERR_TIMEOUT = 7     /* a bounded wait inside a kernel ran out.  The sample concerned is skipped: no loss, no
                                gradient.  If the wait that ran out was for rows of W2, the sample's rows had
                                been handed to the update already: they receive an Adam update with a zero
                                gradient from this sample (their moments decay), unlike rows nobody touched.    */
} dslide_status;

enum { DSLIDE_SIMHASH = 0, DSLIDE_DWTA = 1 };

typedef struct {
  int32_t input_dim, hidden_dim, output_dim; /* D, H, N.  H must be a multiple of 4 and at most 1024.          */
  int32_t hash_family;                       /* DSLIDE_SIMHASH (sparse +1/-1 projections) or DSLIDE_DWTA        */
  int32_t K, L;                              /* K hash functions per table, L tables (Section 4.1)              */
  int32_t dwta_bin_size;                     /* power of two, divides H; 0 means 8                              */
  int32_t srp_nnz;                           /* nonzeros per SimHash projection; 0 means ceil(H/3)              */
  int32_t bucket_cap;                        /* a query reads at most this many (lowest) ids of a bucket        */
  int32_t rebuild_period0;                   /* first scheduled rebuild after this many steps; 0 = never        */
  float rebuild_growth_lambda;               /* later gaps: max(1, floor(period0 * exp(lambda * rebuilds)))     */
  int32_t redraw_hash_fns;                   /* 1: draw new hash functions at every rebuild (Algorithm 1)       */
  int32_t force_dense;                       /* 1: every output neuron is active, no hashing (Section 3.6)      */
  int32_t max_batch;                         /* largest batch a call may pass (at most 4096)                    */
  int32_t max_labels;                        /* largest label list of one sample                                */
  int32_t max_active_per_sample;             /* 0 means L * bucket_cap + max_labels (N when force_dense)        */
  float lr, beta1, beta2, eps;               /* Adam (Section 4.1: 1e-4, 0.9, 0.999, 1e-8)                      */
  float init_std;                            /* weights ~ N(0, init_std^2); biases and moments start at 0       */
  uint64_t seed;
  int32_t device;                            /* CUDA device ordinal                                             */
  int32_t dedup_mode;                        /* 0 auto; 1 bitmap in shared memory; 2 sort in shared memory      */
  void* stream;                              /* cudaStream_t the context enqueues on (NULL = default stream)    */
  int32_t dwta_densify;                      /* 1: DWTA densification for queries (Section 4.1 names the family):
                                                a bin of the hidden activation whose values are all zero borrows
                                                the position of the first non-empty bin along a seeded probe
                                                sequence of 16 other functions (0 when all are empty); 0: such a
                                                bin yields position 0.  Weight rows are never densified.          */
  int32_t sample_budget;                     /* Section 3.7: active neurons kept per sample, the sample's labels
                                                included; when more are retrieved, reservoir sampling (draws
                                                numbered by step, sample and candidate) keeps budget - labels of
                                                the others; fewer are left as they are.  0 = no budget.  The
                                                work space must fit the forward kernel's shared memory: about
                                                5 * (L * bucket_cap) + 8 * budget bytes <= 64 KB, else
                                                dslide_init returns DSLIDE_ERR_INVALID_ARG.                       */
  int32_t budget_fill;                       /* 1 (needs sample_budget > 0 and max_active_per_sample = 0): a
                                                sample whose retrieved neurons and labels are fewer than the
                                                budget is topped up with uniformly drawn neurons (Section 3.7):
                                                ids drawn one after the other, repeats and members passed over,
                                                until min(budget, N) members or 2 * missing + 64 draws.  The
                                                per-sample arrays then hold up to budget entries; the work space
                                                (about 80 bytes per budgeted neuron) must fit the forward
                                                kernel's shared memory, else DSLIDE_ERR_INVALID_ARG.              */
  int32_t inputs_ready;                      /* dslide_train_step only.  0: the batch arrays may still be written by
                                                work enqueued earlier on the context's stream (a kernel or copy of
                                                the caller's); the step reads them only after that work has
                                                completed.  1: the caller promises that the five arrays were
                                                complete in device memory BEFORE the call (their producer has
                                                finished, not merely been enqueued); the step then reads them while
                                                the previous step's update is still draining, which shortens the
                                                step by a few microseconds.  The host-buffer entry points wait for
                                                their own copy and always read early.                              */
  int32_t hidden_K, hidden_L, hidden_cap;    /* LSH-sampled hidden layer (Algorithm 1 retrieves the active neurons
                                                of EVERY layer; Section 3.6: the dense layer is the case "sparsity
                                                is 1").  hidden_L = 0: dense hidden layer.  hidden_L > 0: hidden_L
                                                tables of hidden_K-bit sparse-random-projection codes over the hidden
                                                neurons' weight vectors (columns of W1), queried with the sparse
                                                input; a query reads at most hidden_cap ids of a bucket.  A neuron
                                                that is not retrieved has activation 0, passes no gradient on, and
                                                only weights W1[c][k] with input c nonzero and neuron k retrieved
                                                (for some sample of the batch) are updated; likewise the bias of k.
                                                Entry (c, p) of the projections: +1, -1, 0 with probability 1/6,
                                                1/6, 2/3, drawn per entry.  hidden_K <= 16, hidden_L <= 64,
                                                hidden_K * hidden_L <= 256.  Rebuilt with the output layer's tables. */
} dslide_config;

/* Tensors readable and writable through dslide_get_tensor / dslide_set_tensor. */
enum {
  DSLIDE_T_W1 = 0, DSLIDE_T_B1, DSLIDE_T_W2, DSLIDE_T_B2,          /* f32 [D*H], [H], [N*H], [N]                */
  DSLIDE_T_M_W1, DSLIDE_T_V_W1, DSLIDE_T_M_B1, DSLIDE_T_V_B1,      /* Adam first / second moments (Section 3.5) */
  DSLIDE_T_M_W2, DSLIDE_T_V_W2, DSLIDE_T_M_B2, DSLIDE_T_V_B2,
  DSLIDE_T_HASH_IDX,    /* i32 [K*L][srp_nnz] (SimHash, ascending per projection) or [K*L][bin] (DWTA)          */
  DSLIDE_T_HASH_SIGN,   /* i32 [K*L][srp_nnz], +1 / -1 (SimHash only; 0 bytes for DWTA)                         */
  DSLIDE_T_BUCKET_OFF,  /* i32 [L][2^bits + 1], bits = K (SimHash) or K*log2(bin) (DWTA)                        */
  DSLIDE_T_BUCKET_IDS,  /* i32 [L][N]: per table, neuron ids grouped by bucket, ascending inside a bucket       */
  DSLIDE_T_COUNTERS,    /* i64 [3]: Adam step count t, rebuild count r, step of the next scheduled rebuild      */
  DSLIDE_T_PROJ1,       /* i8 [D][hidden_K * hidden_L]: the hidden layer's projections (+1 / -1 / 0); 0 bytes when dense */
  DSLIDE_T_BUCKET1_OFF, /* i32 [hidden_L][2^hidden_K + 1]                                                        */
  DSLIDE_T_BUCKET1_IDS, /* i32 [hidden_L][H]: hidden neuron ids grouped by bucket, ascending inside a bucket     */
  DSLIDE_T_COUNT
};

/* Per-sample snapshot of the last dslide_train_step (Section 3.6), for dslide_get_last. */
enum {
  DSLIDE_LAST_HIDDEN = 0, /* f32 [B][H]                                                        */
  DSLIDE_LAST_CODES,      /* u32 [B][L] bucket codes of the hidden activations                  */
  DSLIDE_LAST_ACT_COUNT,  /* i32 [B] size of each active set                                    */
  DSLIDE_LAST_ACT_IDS,    /* i32 [B][stride] ascending ids, first count[s] entries valid        */
  DSLIDE_LAST_ACT_LOGIT,  /* f32 [B][stride]                                                    */
  DSLIDE_LAST_ACT_PROB,   /* f32 [B][stride] softmax over the active set                        */
  DSLIDE_LAST_ACT_ERR,    /* f32 [B][stride] (p - [label]/|labels|) / B                         */
  DSLIDE_LAST_LOSS,       /* f32 [B]                                                            */
  DSLIDE_LAST_DHIDDEN,    /* f32 [B][H] error back-propagated to the hidden layer               */
  DSLIDE_LAST_CODES1,     /* u32 [B][hidden_L] bucket codes of the inputs (sampled hidden layer)  */
  DSLIDE_LAST_HIDDEN_MASK,/* u32 [B][ceil(H/32)] bit k = hidden neuron k active for the sample    */
  DSLIDE_LAST_COUNT
};

/* Algorithm 1, initialisation: allocates the model, draws the weights and the hash
 * functions of rebuild count 0 and indexes every output neuron into the L tables
 * (Section 2.1, phase 1).  Synchronous.  *out receives the context. */
dslide_status dslide_init(const dslide_config* cfg, dslide_ctx** out);

/* Frees everything the context owns after draining its stream.  Synchronous. */
dslide_status dslide_destroy(dslide_ctx* ctx);

/* Algorithm 1 "Rebuild hash tables and hash functions", outside the schedule: the
 * rebuild count goes up by one, new functions are drawn when redraw_hash_fns is
 * set, and every neuron's current weight row is hashed into the tables again. */
dslide_status dslide_rebuild_tables(dslide_ctx* ctx);

/* Hash the tables again with the hash functions currently loaded and the current
 * weights; the rebuild count does not change.  For callers that load their own
 * hash functions or weights with dslide_set_tensor. */
dslide_status dslide_build_tables(dslide_ctx* ctx);

/* One training step on one batch (Algorithm 1, inner loops and the Adam line; Section
 * 2.1 feed-forward and back-propagation stages):
 *   hidden layer from the CSR rows -> L bucket codes -> union of the retrieved buckets
 *   plus the sample's labels -> logits and softmax over that set only -> errors ->
 *   sparse back-propagation -> Adam on the touched rows of W2, b2, W1 and on b1 ->
 *   the scheduled rebuild if this step is due.
 * batch in [1, max_batch].  CSR: row_ptr[batch+1] (row_ptr[0] = 0, non-decreasing),
 * col_idx / vals [row_ptr[batch]], column ids in [0, D), ascending inside a row.
 * Labels: label_ptr[batch+1], labels[label_ptr[batch]], ids in [0, N), at least one and
 * at most max_labels per sample; duplicates inside a sample count once.
 * All five are device pointers.  loss_out: device float, may be NULL; receives the mean
 * loss of the batch.  The loss of sample s is -(1/|Y_s|) sum_{y in Y_s} log p_y with p
 * the softmax over the active set. */
dslide_status dslide_train_step(dslide_ctx* ctx, int32_t batch, const int32_t* row_ptr,
                                const int32_t* col_idx, const float* vals,
                                const int32_t* label_ptr, const int32_t* labels, float* loss_out);

/* The same step for callers whose batch lives in HOST memory: copies the five arrays to
 * the device (nnz = row_ptr[batch] and label_ptr[batch] are read on the host), runs the
 * step, copies the mean loss back to *loss_out (host, may be NULL) and waits for it.
 * Returns the sticky device status like dslide_sync. */
dslide_status dslide_train_step_host(dslide_ctx* ctx, int32_t batch, const int32_t* row_ptr,
                                     const int32_t* col_idx, const float* vals,
                                     const int32_t* label_ptr, const int32_t* labels,
                                     float* loss_out);

/* The same step, pipelined: the call packs and enqueues this batch and returns as soon as the PREVIOUS
 * host-buffer step has reported -- its loss and status are known, its weight update may still be running --
 * handing out that step's mean loss (*prev_loss_out, may be NULL) and sticky status (the return value);
 * *have_prev (may be NULL) tells whether there was a previous step to report.
 * The device therefore always has one step queued while the host prepares the next.  The arrays are copied
 * into the library's pinned buffer before the call returns, so the caller may reuse them at once.
 * dslide_host_result waits for the newest pipelined step and hands out its loss and status (*have = 0 and
 * DSLIDE_OK when none is outstanding) and, like dslide_sync, clears the sticky status; between those calls a
 * status seen by one step is reported by the following steps as well.  dslide_train_step_host may be mixed in
 * (it drops uncollected results). */
dslide_status dslide_train_step_host_async(dslide_ctx* ctx, int32_t batch, const int32_t* row_ptr,
                                           const int32_t* col_idx, const float* vals, const int32_t* label_ptr,
                                           const int32_t* labels, float* prev_loss_out, int32_t* have_prev);
dslide_status dslide_host_result(dslide_ctx* ctx, float* loss_out, int32_t* have);

/* Inference: hidden layer -> codes -> retrieved set (dense = 0) or every neuron
 * (dense = 1) -> logits -> the k largest by (logit descending, id ascending).
 * out_ids [batch*k] (device, -1 where fewer than k candidates), out_scores [batch*k]
 * (device, -inf there).  1 <= k <= 64.  The paper reports accuracy but not how it
 * evaluates; this is the reading taken.  With dense = 1 the first call (and any call
 * with a larger batch * k) allocates device work space for the partial lists after
 * waiting for the stream.  With dense = 1, k <= 8 and a hidden width that is a multiple of
 * 32 up to 256 the scores of all neurons are first taken on the tensor pipe in TF32 and
 * used as a filter only: the candidates are re-scored in fp32, and a sample for which
 * the filter cannot be shown to be exact (an error bound on the TF32 scores decides) is
 * scored over all neurons in fp32, so the results are those of the fp32 path.  A predict call uses the per-sample work space of the training
 * step: afterwards the snapshot read by dslide_get_last (hidden activations with dense = 1;
 * active ids and logits with dense = 0, whose counts, codes and losses still belong to the
 * last training step) is no longer that of the last training step.  The next training step
 * rewrites all of it. */
dslide_status dslide_predict_topk(dslide_ctx* ctx, int32_t batch, const int32_t* row_ptr,
                                  const int32_t* col_idx, const float* vals, int32_t k,
                                  int32_t dense, int32_t* out_ids, float* out_scores);

/* Waits for the context's stream; returns and clears the sticky device status. */
dslide_status dslide_sync(dslide_ctx* ctx);

/* State I/O (check-pointing and the parity harness).  Synchronous.  host pointers.
 * nbytes must equal the tensor's size exactly.  Setting weights or hash functions does
 * not rebuild the tables; call dslide_build_tables. */
enum { DSLIDE_DT_F32 = 0, DSLIDE_DT_I32 = 1, DSLIDE_DT_I64 = 2, DSLIDE_DT_I8 = 3 };
dslide_status dslide_tensor_info(dslide_ctx* ctx, int32_t which, int64_t* nbytes, int32_t* dtype /* may be NULL: DSLIDE_DT_* */);
dslide_status dslide_get_tensor(dslide_ctx* ctx, int32_t which, void* host_dst, int64_t nbytes);
dslide_status dslide_set_tensor(dslide_ctx* ctx, int32_t which, const void* host_src, int64_t nbytes);

/* Snapshot of the last training step.  Synchronous.  host_dst receives min(nbytes,
 * size) bytes; *stride (may be NULL) receives the row stride, in elements, of the
 * per-sample active arrays. */
dslide_status dslide_last_info(dslide_ctx* ctx, int32_t which, int64_t* nbytes, int32_t* stride);
dslide_status dslide_get_last(dslide_ctx* ctx, int32_t which, void* host_dst, int64_t nbytes);

/* Per-step statistics of the last training step, read from the device.  Synchronous.
 * out[0] = sum of active-set sizes, out[1] = distinct touched rows of W2, out[2] =
 * distinct touched rows of W1, out[3] = nonzeros in the batch. */
dslide_status dslide_last_stats(dslide_ctx* ctx, int64_t out[4]);

/* Totals since the last reset, read from the device.  Synchronous.  out[0] = training steps,
 * out[1] = sum of active-set sizes, out[2] = sum of distinct touched W2 rows, out[3] = sum of
 * distinct touched W1 rows, out[4] = nonzeros, out[5] = bucket entries read by the lookups.
 * reset != 0 clears the totals afterwards. */
dslide_status dslide_cum_stats(dslide_ctx* ctx, int64_t out[6], int32_t reset);

/* Per-kernel device time.  Between dslide_profile_begin and dslide_profile_end every kernel the
 * context launches is bracketed by a CUDA event pair on the context's stream; dslide_profile_end
 * waits for the stream and returns, per kernel, the summed milliseconds and the launch count.
 * The event records add a little latency between kernels: use it to split time between kernels,
 * not for the throughput figure. */
enum {
  DSLIDE_K_FORWARD = 0, DSLIDE_K_ADAM_DENSE, DSLIDE_K_ADAM, DSLIDE_K_DRAW_HASH, DSLIDE_K_HASH_NEURONS,
  DSLIDE_K_BUCKET_SCAN, DSLIDE_K_SORT_HIST, DSLIDE_K_SORT_SCAN, DSLIDE_K_SORT_SCATTER,
  DSLIDE_K_PREDICT, DSLIDE_K_INIT, DSLIDE_K_PLACE_IDS, DSLIDE_K_ORDER_BUCKETS, DSLIDE_K_COUNT
};
dslide_status dslide_profile_begin(dslide_ctx* ctx);
dslide_status dslide_profile_end(dslide_ctx* ctx, double ms[DSLIDE_K_COUNT], int64_t launches[DSLIDE_K_COUNT]);

/* Bucket sort of one hash table for callers that must not allocate.  (The paper has no
 * counterpart: this is a packaging variant of the table build's sort, not a step of the method.)
 *
 * Who needs it: code that reaches this library from a place where device allocation is off
 * limits -- a plug-in that is only handed buffers, a service that has promised a fixed memory
 * footprint, a caller running inside somebody else's memory pool.  This call makes no
 * cudaMalloc / cudaFree and calls nothing that allocates; it needs no dslide_ctx.  Its work
 * space is a static device array inside the library image: every GPU that loads libdslide.so
 * holds those DSLIDE_STATIC_SORT_MAX_N * 8 bytes (2 MiB) until the process exits.
 *
 * codes[n] (device): bucket code of neuron i in this table; only the low `bits` bits are used.
 * Output (device, caller-owned): bucket_off[2^bits + 1] = where each bucket starts in
 * bucket_ids (bucket_off[0] = 0, bucket_off[2^bits] = n); bucket_ids[n] = the ids 0..n-1
 * grouped by code, ascending inside a bucket -- the layout of one table of
 * DSLIDE_T_BUCKET_OFF / DSLIDE_T_BUCKET_IDS.  Both outputs are fully overwritten.
 * Limits: 0 <= n <= DSLIDE_STATIC_SORT_MAX_N and 1 <= bits <= DSLIDE_STATIC_SORT_MAX_BITS,
 * otherwise DSLIDE_ERR_OVERFLOW and nothing is launched.
 * Runs as one thread block on `stream` (a cudaStream_t, NULL = default stream) of the CURRENT
 * device, asynchronously.  The first call on each device looks up the array's device address
 * (once per device, with that device current); make that first call before any stream capture.
 * All calls on a device share the one array, which keeps the last call's contents: the kernel
 * overwrites what it reads, but two calls that overlap on the GPU (different streams, no
 * ordering between them) race on it -- order them.  The address looked up by the first call is
 * kept per device ordinal for the life of the process: it is stale after cudaDeviceReset, and
 * the first call on a device must not race with another first call from a second host thread. */
#define DSLIDE_STATIC_SORT_MAX_N 262144
#define DSLIDE_STATIC_SORT_MAX_BITS 18
dslide_status dslide_bucket_sort_static(const uint32_t* codes, int32_t n, int32_t bits,
                                        int32_t* bucket_off, int32_t* bucket_ids, void* stream);

/* Number of kernels the context has launched since dslide_init. */
int64_t dslide_kernel_launches(const dslide_ctx* ctx);

const char* dslide_status_str(dslide_status s);

#ifdef __cplusplus
}
#endif
#endif /* DSLIDE_H */
