// The C ABI of libdslide (include/dslide.h): context life cycle, argument checks, the rebuild
// schedule (Section 3.1; Algorithm 1 places the rebuild after the weight update), state I/O.
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <atomic>
#include <vector>

#include "common.cuh"

namespace dslide {
int sort_tile_elems();
int sort_max_width();
int bucket_scan_chunk();
int order_small_max();
int order_block_max();
}

using namespace dslide;

struct dslide_ctx { Ctx c; };

namespace dslide {
struct ProfRec { int kid; cudaEvent_t beg, end; };

LaunchScope::LaunchScope(Ctx* c_, int kid_) : c(c_), kid(kid_), rec(-1) {
  c->launches++;
  if (!c->profiling || !c->prof) return;
  auto* v = static_cast<std::vector<ProfRec>*>(c->prof);
  ProfRec r;
  r.kid = kid;
  if (cudaEventCreate(&r.beg) != cudaSuccess) return;
  if (cudaEventCreate(&r.end) != cudaSuccess) { cudaEventDestroy(r.beg); return; }
  cudaEventRecord(r.beg, c->stream);
  v->push_back(r);
  rec = (long long)v->size() - 1;      // an index, not a pointer: the vector may grow (and move) before the scope ends
}
LaunchScope::~LaunchScope() {
  if (rec < 0 || !c->prof) return;
  auto* v = static_cast<std::vector<ProfRec>*>(c->prof);
  if ((size_t)rec < v->size()) cudaEventRecord((*v)[(size_t)rec].end, c->stream);
}
}  // namespace dslide

namespace {

#define CU(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return e_ == cudaErrorMemoryAllocation ? DSLIDE_ERR_OOM : DSLIDE_ERR_CUDA; } while (0)

template <typename T>
cudaError_t dalloc(T** p, size_t n, cudaStream_t st, bool zero) {
  *p = nullptr;
  if (n == 0) n = 1;
  cudaError_t e = cudaMalloc((void**)p, n * sizeof(T));
  if (e != cudaSuccess) return e;
  if (zero) e = cudaMemsetAsync(*p, 0, n * sizeof(T), st);
  return e;
}

void free_all(Ctx* c) {
  void* ptrs[] = {c->W1, c->b1, c->W2, c->hdr1, c->hdr2, c->mW1, c->vW1, c->mb1, c->vb1, c->mW2, c->vW2,
                  c->hash_idx, c->hash_sign, c->bucket_off, c->bucket_ids, c->h, c->dh, c->loss, c->codes,
                  c->act_cnt, c->act_ids, c->act_z, c->act_p, c->act_g, c->mask1, c->ovf1, c->ovf2, c->hotmap1, c->hotcoef1,
                  c->mask2, c->proj1, c->bucket1_off, c->bucket1_ids, c->codes1n, c->codes1, c->hmask, c->cmask1, c->own1, c->own2, c->hot_rows, c->med_rows, c->hot_part, c->hot_done, c->dstate, c->keysA, c->keysB, c->valsA, c->valsB, c->tile_hist, c->bucket_part, c->ord_mid, c->ord_big, c->ord_cnt,
                  c->st_dev[0], c->st_dev[1], c->st_dev[2], c->pd_part};
  for (void* p : ptrs) if (p) cudaFree(p);
  for (int b = 0; b < ST_SETS; ++b) {
    if (c->st_host[b]) cudaFreeHost(c->st_host[b]);
    if (c->st_res[b]) cudaFreeHost(c->st_res[b]);
    if (c->st_in[b]) cudaEventDestroy(c->st_in[b]);
  }
  if (c->st_copy_in) cudaStreamDestroy(c->st_copy_in);
  if (c->prof) {
    auto* v = static_cast<std::vector<ProfRec>*>(c->prof);
    for (auto& r : *v) { cudaEventDestroy(r.beg); cudaEventDestroy(r.end); }
    delete v;
    c->prof = nullptr;
  }
}

int ilog2_exact(int x) {
  int l = 0;
  while ((1 << l) < x) ++l;
  return (1 << l) == x ? l : -1;
}

struct TensorRef { void* ptr; int64_t bytes; int64_t pitch; };     // pitch != 0: one float every `pitch` bytes

TensorRef tensor_ref(Ctx* c, int which) {
  const int64_t D = c->D, H = c->H, N = c->N, f = sizeof(float);
  switch (which) {
    case DSLIDE_T_W1: return {c->W1, D * H * f};
    case DSLIDE_T_B1: return {c->b1, H * f};
    case DSLIDE_T_W2: return {c->W2, N * H * f};
    case DSLIDE_T_B2: return {&c->hdr2->b, N * f, (int64_t)sizeof(RowHdr)};
    case DSLIDE_T_M_W1: return {c->mW1, D * H * f};
    case DSLIDE_T_V_W1: return {c->vW1, D * H * f};
    case DSLIDE_T_M_B1: return {c->mb1, H * f};
    case DSLIDE_T_V_B1: return {c->vb1, H * f};
    case DSLIDE_T_M_W2: return {c->mW2, N * H * f};
    case DSLIDE_T_V_W2: return {c->vW2, N * H * f};
    case DSLIDE_T_M_B2: return {&c->hdr2->mb, N * f, (int64_t)sizeof(RowHdr)};
    case DSLIDE_T_V_B2: return {&c->hdr2->vb, N * f, (int64_t)sizeof(RowHdr)};
    case DSLIDE_T_HASH_IDX: return {c->hash_idx, (int64_t)c->KL * c->fn_len * 4};
    case DSLIDE_T_HASH_SIGN: return {c->hash_sign, c->cfg.hash_family == DSLIDE_SIMHASH ? (int64_t)c->KL * c->fn_len * 4 : 0};
    case DSLIDE_T_BUCKET_OFF: return {c->bucket_off, (int64_t)c->L * (c->nb + 1) * 4};
    case DSLIDE_T_BUCKET_IDS: return {c->bucket_ids, (int64_t)c->L * N * 4};
    case DSLIDE_T_COUNTERS: return {nullptr, 3 * 8};
    case DSLIDE_T_PROJ1: return {c->proj1, c->L1 > 0 ? D * c->KL1 : 0};
    case DSLIDE_T_BUCKET1_OFF: return {c->bucket1_off, c->L1 > 0 ? (int64_t)c->L1 * (((int64_t)1 << c->K1) + 1) * 4 : 0};
    case DSLIDE_T_BUCKET1_IDS: return {c->bucket1_ids, c->L1 > 0 ? (int64_t)c->L1 * H * 4 : 0};
  }
  return {nullptr, -1};
}

dslide_status drain(Ctx* c) {
  CU(cudaStreamSynchronize(c->stream));
  return DSLIDE_OK;
}

dslide_status rebuild(Ctx* c, bool bump) {
  if (bump) {
    c->r_host += 1;
    if (c->cfg.redraw_hash_fns) {
      if (!c->dense) CU(launch_draw_hash(c, c->r_host));
      CU(launch_draw_proj1(c, c->r_host));
    }
  }
  if (!c->dense) CU(launch_build_tables(c));
  CU(launch_build_tables1(c));        // the hidden layer's tables, when it is LSH-sampled
  return DSLIDE_OK;
}

}  // namespace

extern "C" {

const char* dslide_status_str(dslide_status s) {
  switch (s) {
    case DSLIDE_OK: return "ok";
    case DSLIDE_ERR_INVALID_ARG: return "invalid argument";
    case DSLIDE_ERR_OOM: return "out of device memory";
    case DSLIDE_ERR_CUDA: return "CUDA error";
    case DSLIDE_ERR_OVERFLOW: return "active set, label list or batch exceeds the configured maximum";
    case DSLIDE_ERR_BAD_INDEX: return "feature or label id out of range, or columns not ascending";
    case DSLIDE_ERR_STATE: return "call not valid in this state";
    case DSLIDE_ERR_TIMEOUT: return "timeout";
  }
  return "unknown status";
}

dslide_status dslide_init(const dslide_config* cfg, dslide_ctx** out) {
  if (!cfg || !out) return DSLIDE_ERR_INVALID_ARG;
  *out = nullptr;
  dslide_config k = *cfg;
  if (k.input_dim < 1 || k.hidden_dim < 4 || k.hidden_dim > 1024 || (k.hidden_dim & 3) || k.output_dim < 1)
    return DSLIDE_ERR_INVALID_ARG;
  if (k.hash_family != DSLIDE_SIMHASH && k.hash_family != DSLIDE_DWTA) return DSLIDE_ERR_INVALID_ARG;
  if (k.K < 1 || k.L < 1 || k.L > 1024 || k.bucket_cap < 1) return DSLIDE_ERR_INVALID_ARG;
  if (k.max_batch < 1 || k.max_batch > 4096 || k.max_labels < 1 || k.max_labels > 4096) return DSLIDE_ERR_INVALID_ARG;
  if (!(k.lr > 0.f) || !(k.beta1 >= 0.f && k.beta1 < 1.f) || !(k.beta2 >= 0.f && k.beta2 < 1.f) || !(k.eps > 0.f))
    return DSLIDE_ERR_INVALID_ARG;
  if (k.rebuild_period0 < 0 || k.init_std < 0.f || k.dedup_mode < 0 || k.dedup_mode > 2) return DSLIDE_ERR_INVALID_ARG;
  if (k.dwta_densify < 0 || k.dwta_densify > 1 || k.sample_budget < 0) return DSLIDE_ERR_INVALID_ARG;
  if (k.budget_fill < 0 || k.budget_fill > 1 || k.inputs_ready < 0 || k.inputs_ready > 1) return DSLIDE_ERR_INVALID_ARG;
  if (k.hidden_L < 0 || k.hidden_L > 64) return DSLIDE_ERR_INVALID_ARG;
  if (k.hidden_L > 0 && (k.hidden_K < 1 || k.hidden_K > 16 || k.hidden_K * k.hidden_L > 256 || k.hidden_cap < 1)) return DSLIDE_ERR_INVALID_ARG;
  if (k.budget_fill && (k.sample_budget < 1 || k.max_active_per_sample != 0 || k.force_dense)) return DSLIDE_ERR_INVALID_ARG;
  if (k.dwta_bin_size == 0) k.dwta_bin_size = 8;
  if (k.srp_nnz == 0) k.srp_nnz = (k.hidden_dim + 2) / 3;
  int lg_bin = 0, bits = 0, fn_len = 0;
  if (k.hash_family == DSLIDE_DWTA) {
    lg_bin = ilog2_exact(k.dwta_bin_size);
    if (lg_bin < 1 || k.dwta_bin_size > 256 || k.hidden_dim % k.dwta_bin_size) return DSLIDE_ERR_INVALID_ARG;
    bits = k.K * lg_bin;
    fn_len = k.dwta_bin_size;
  } else {
    if (k.srp_nnz < 1 || k.srp_nnz > k.hidden_dim) return DSLIDE_ERR_INVALID_ARG;
    bits = k.K;
    fn_len = k.srp_nnz;
  }
  if (bits > 24 || (int64_t)k.K * k.L > 65536) return DSLIDE_ERR_INVALID_ARG;
  if ((int64_t)k.L * k.output_dim >= (int64_t)1 << 31) return DSLIDE_ERR_INVALID_ARG;
  int64_t act_stride = k.force_dense ? k.output_dim
                       : (k.max_active_per_sample > 0 ? k.max_active_per_sample
                                                      : (int64_t)k.L * k.bucket_cap + k.max_labels);
  if (!k.force_dense && act_stride > (int64_t)k.L * k.bucket_cap + k.max_labels)
    act_stride = (int64_t)k.L * k.bucket_cap + k.max_labels;
  if (k.budget_fill && act_stride < k.sample_budget) act_stride = k.sample_budget;     // a filled set has up to budget members
  if (act_stride > k.output_dim) act_stride = k.output_dim;
  if (act_stride < 1) return DSLIDE_ERR_INVALID_ARG;

  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || k.device < 0 || k.device >= ndev) return DSLIDE_ERR_CUDA;
  CU(cudaSetDevice(k.device));

  dslide_ctx* h = new (std::nothrow) dslide_ctx;
  if (!h) return DSLIDE_ERR_OOM;
  memset(h, 0, sizeof(*h));
  Ctx* c = &h->c;
  c->cfg = k;
  c->D = k.input_dim; c->H = k.hidden_dim; c->N = k.output_dim; c->K = k.K; c->L = k.L; c->KL = k.K * k.L;
  c->bits = bits; c->lg_bin = lg_bin; c->fn_len = fn_len; c->cap = k.bucket_cap;
  c->nb = (int64_t)1 << bits;
  c->act_stride = (int)act_stride;
  c->Wd = (k.max_batch + 31) / 32;
  c->L1 = k.hidden_L; c->K1 = k.hidden_L > 0 ? k.hidden_K : 0; c->KL1 = c->K1 * c->L1; c->cap1 = k.hidden_cap;
  c->Hw = (k.hidden_dim + 31) / 32;
  c->dense = k.force_dense ? 1 : 0;
  c->stream = (cudaStream_t)k.stream;
  c->next_rebuild = k.rebuild_period0;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, k.device) != cudaSuccess) { delete h; return DSLIDE_ERR_CUDA; }
  c->num_sms = prop.multiProcessorCount;

  // radix sort geometry
  c->sort_passes = (bits + sort_max_width() - 1) / sort_max_width();
  c->sort_width = (bits + c->sort_passes - 1) / c->sort_passes;
  c->sort_tiles = (c->N + sort_tile_elems() - 1) / sort_tile_elems();

  const size_t D = c->D, H = c->H, N = c->N, B = k.max_batch, S = c->act_stride;
  cudaStream_t st = c->stream;
  cudaError_t e = cudaSuccess;
#define A(ptr, n, zero) if (e == cudaSuccess) e = dalloc(&c->ptr, (size_t)(n), st, zero)
  A(W1, D * H, false); A(mW1, D * H, true); A(vW1, D * H, true);
  A(b1, H, true); A(mb1, H, true); A(vb1, H, true);
  A(W2, N * H, false); A(mW2, N * H, true); A(vW2, N * H, true);
  A(hdr2, N, true);
  A(hash_idx, (size_t)c->KL * fn_len, true); A(hash_sign, (size_t)c->KL * fn_len, true);
  A(h, B * H, true); A(dh, B * H, true); A(loss, B, true); A(codes, B * c->L, true);
  A(act_cnt, B, true); A(act_z, B * S, true); A(act_p, B * S, true); A(act_g, B * S, true);
  A(hdr1, D, true); A(mask1, D * c->Wd, true); A(own1, D, true); A(ovf1, D * PAIR_T, false);
  A(hot_rows, HOT_CAP, true); A(med_rows, MED_CAP, true); A(hot_done, HOT_CAP, true); A(hot_part, (size_t)HOT_CAP * HOT_SLICES * (H + 4), true);
  A(dstate, 1, true);
  A(hotmap1, D, false); A(hotcoef1, (size_t)HOTMAP_CAP * B, false);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->hotmap1, 0xff, D * sizeof(int32_t), st);
  if (c->L1 > 0) {
    A(proj1, D * (size_t)c->KL1, true);
    A(bucket1_off, (size_t)c->L1 * (((size_t)1 << c->K1) + 1), true); A(bucket1_ids, (size_t)c->L1 * H, true);
    A(codes1n, (size_t)c->L1 * H + ((size_t)c->KL1 * H + 3) / 4 + 1, true);     // codes, then one byte per (projection, neuron)
    A(codes1, B * (size_t)c->L1, true); A(hmask, B * (size_t)c->Hw, true); A(cmask1, D * (size_t)c->Hw, true);
  }
  if (!c->dense) {
    A(act_ids, B * S, true);
    A(mask2, N * c->Wd, true);
    A(ovf2, N * PAIR_T, false);
    A(own2, N, true);
    A(bucket_off, (size_t)c->L * (size_t)(c->nb + 1), true); A(bucket_ids, (size_t)c->L * N, true);
    A(keysA, (size_t)c->L * N, false);
    // codes wider than one radix digit: every id is placed at its bucket's start plus its rank of arrival there and the
    // large buckets are ordered afterwards, no radix passes
    c->place_path = c->bits > sort_max_width() ? 1 : 0;
    if (c->place_path) {
      A(keysB, (size_t)c->L * N, false);      // here: the rank of every id inside its bucket
      A(ord_mid, (size_t)c->L * (N / (order_small_max() + 1) + 1), false);
      A(ord_big, (size_t)c->L * (N / (order_block_max() + 1) + 1), false);
      A(ord_cnt, 2, true);
    } else {
      if (c->sort_passes > 1) { A(keysB, (size_t)c->L * N, false); A(valsA, (size_t)c->L * N, false); }
      if (c->sort_passes > 2) { A(valsB, (size_t)c->L * N, false); }
      A(tile_hist, (size_t)c->L * ((size_t)1 << c->sort_width) * c->sort_tiles, false);
    }
    A(bucket_part, (size_t)c->L * (size_t)((c->nb + 1 + bucket_scan_chunk() - 1) / bucket_scan_chunk()), false);
  }
#undef A
  for (int b = 0; b < ST_SETS; ++b) {
    if (e == cudaSuccess) e = cudaHostAlloc((void**)&c->st_res[b], sizeof(HostResult), cudaHostAllocMapped);
    if (e == cudaSuccess) {
      memset(c->st_res[b], 0, sizeof(HostResult));
      e = cudaHostGetDevicePointer((void**)&c->st_res_dev[b], c->st_res[b], 0);
    }
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->st_in[b], cudaEventDisableTiming);
  }
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->st_copy_in, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = setup_forward(c);
  if (e == cudaSuccess) e = launch_init_gauss(c, c->W1, (int64_t)(D * H), RNG_W1);
  if (e == cudaSuccess) e = launch_init_gauss(c, c->W2, (int64_t)(N * H), RNG_W2);
  if (e == cudaSuccess && !c->dense) e = launch_draw_hash(c, 0);
  if (e == cudaSuccess && !c->dense) e = launch_build_tables(c);
  if (e == cudaSuccess) e = launch_draw_proj1(c, 0);
  if (e == cudaSuccess) e = launch_build_tables1(c);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) {
    dslide_status s = e == cudaErrorMemoryAllocation ? DSLIDE_ERR_OOM
                      : e == cudaErrorInvalidValue ? DSLIDE_ERR_INVALID_ARG : DSLIDE_ERR_CUDA;
    cudaGetLastError();
    free_all(c);
    delete h;
    return s;
  }
  *out = h;
  return DSLIDE_OK;
}

dslide_status dslide_destroy(dslide_ctx* ctx) {
  if (!ctx) return DSLIDE_ERR_INVALID_ARG;
  cudaSetDevice(ctx->c.cfg.device);
  cudaStreamSynchronize(ctx->c.stream);
  free_all(&ctx->c);
  delete ctx;
  return DSLIDE_OK;
}

dslide_status dslide_rebuild_tables(dslide_ctx* ctx) {
  if (!ctx) return DSLIDE_ERR_INVALID_ARG;
  return rebuild(&ctx->c, true);
}

dslide_status dslide_build_tables(dslide_ctx* ctx) {
  if (!ctx) return DSLIDE_ERR_INVALID_ARG;
  return rebuild(&ctx->c, false);
}

namespace {

// One step.  With host_res, the update kernel also reports {status, loss, host_seq} into mapped host memory.
dslide_status train_step_impl(dslide_ctx* ctx, int32_t batch, const int32_t* row_ptr, const int32_t* col_idx,
                              const float* vals, const int32_t* label_ptr, const int32_t* labels, float* loss_out,
                              HostResult* host_res, unsigned int host_seq) {
  Ctx* c = &ctx->c;
  // a host-buffer step has waited for its own input copy; a device-pointer step reads early only on the caller's word
  CU(launch_forward_train(c, batch, row_ptr, col_idx, vals, label_ptr, labels, host_res ? 1 : (c->cfg.inputs_ready ? 1 : 0)));
  CU(launch_update(c, batch, row_ptr, col_idx, vals, loss_out, host_res, host_seq));
  c->t_host += 1;
  if (c->cfg.rebuild_period0 > 0 && c->t_host == c->next_rebuild) {
    dslide_status s = rebuild(c, true);
    if (s != DSLIDE_OK) return s;
    double gap = floor((double)c->cfg.rebuild_period0 * exp((double)c->cfg.rebuild_growth_lambda * (double)c->r_host));
    if (gap < 1.0) gap = 1.0;
    c->next_rebuild += (int64_t)gap;
  }
  return DSLIDE_OK;
}

}  // namespace

dslide_status dslide_train_step(dslide_ctx* ctx, int32_t batch, const int32_t* row_ptr, const int32_t* col_idx,
                                const float* vals, const int32_t* label_ptr, const int32_t* labels, float* loss_out) {
  if (!ctx || !row_ptr || !col_idx || !vals || !label_ptr || !labels) return DSLIDE_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (batch < 1) return DSLIDE_ERR_INVALID_ARG;
  if (batch > c->cfg.max_batch) return DSLIDE_ERR_OVERFLOW;
  return train_step_impl(ctx, batch, row_ptr, col_idx, vals, label_ptr, labels, loss_out, nullptr, 0u);
}

namespace {

// Hands out the result of the step that used staging set b: waits until the update kernel of that step has
// written its sequence number into the set's mapped result record, returns the sticky status as it stood at the
// end of that step, stores its mean loss.  The wait polls host memory; every so often it also asks whether the
// stream has gone idle or failed, so that a step that never reports ends the wait with an error.
dslide_status take_result(Ctx* c, int b, float* loss_out) {
  if (!c->st_pending[b]) return DSLIDE_OK;
  c->st_pending[b] = 0;
  volatile HostResult* r = c->st_res[b];
  const unsigned int want = c->st_seq[b];
  for (unsigned long long spins = 1; r->seq != want; ++spins) {
    if ((spins & 0x3ffu) == 0) {
      cudaError_t q = cudaStreamQuery(c->stream);
      if (q == cudaErrorNotReady) continue;
      if (q != cudaSuccess) return DSLIDE_ERR_CUDA;
      if (r->seq != want) return DSLIDE_ERR_CUDA;      // the stream is idle and the step has not reported
    }
  }
  std::atomic_thread_fence(std::memory_order_acquire);
  if (loss_out) *loss_out = r->loss;
  return (dslide_status)r->status;
}

// With the stream drained, a reported status is cleared on the device (as dslide_sync does).
dslide_status drain_and_clear(Ctx* c, dslide_status s) {
  CU(cudaStreamSynchronize(c->stream));
  if (s != DSLIDE_OK) {
    CU(cudaMemsetAsync(&c->dstate->status, 0, sizeof(int), c->stream));
    CU(cudaStreamSynchronize(c->stream));
  }
  return s;
}

// Packs a host batch into staging set b (one pinned buffer, 16-byte aligned pieces), sends it in a single copy
// and enqueues the step.
dslide_status enqueue_host_step(dslide_ctx* ctx, int b, int32_t batch, const int32_t* row_ptr, const int32_t* col_idx,
                                const float* vals, const int32_t* label_ptr, const int32_t* labels) {
  Ctx* c = &ctx->c;
  const int64_t nnz = row_ptr[batch], nlab = label_ptr[batch];
  if (nnz < 0 || nlab < 0 || row_ptr[0] != 0 || label_ptr[0] != 0) return DSLIDE_ERR_INVALID_ARG;
  auto up16 = [](size_t x) { return (x + 15) & ~(size_t)15; };
  const size_t o_rp = 0;
  const size_t o_lp = o_rp + up16(sizeof(int32_t) * ((size_t)batch + 1));
  const size_t o_col = o_lp + up16(sizeof(int32_t) * ((size_t)batch + 1));
  const size_t o_val = o_col + up16(sizeof(int32_t) * (size_t)nnz);
  const size_t o_lab = o_val + up16(sizeof(float) * (size_t)nnz);
  const size_t total = o_lab + up16(sizeof(int32_t) * (size_t)nlab);
  if ((int64_t)total > c->st_cap[b]) {
    CU(cudaStreamSynchronize(c->stream));
    if (c->st_dev[b]) cudaFree(c->st_dev[b]);
    if (c->st_host[b]) cudaFreeHost(c->st_host[b]);
    c->st_dev[b] = nullptr; c->st_host[b] = nullptr; c->st_cap[b] = 0;
    const size_t cap = total + total / 2 + 4096;
    CU(cudaMalloc((void**)&c->st_dev[b], cap));
    CU(cudaMallocHost((void**)&c->st_host[b], cap));
    c->st_cap[b] = (int64_t)cap;
  }
  cudaStream_t st = c->stream;
  unsigned char *hb = c->st_host[b], *db = c->st_dev[b];
  memcpy(hb + o_rp, row_ptr, sizeof(int32_t) * ((size_t)batch + 1));
  memcpy(hb + o_lp, label_ptr, sizeof(int32_t) * ((size_t)batch + 1));
  memcpy(hb + o_col, col_idx, sizeof(int32_t) * (size_t)nnz);
  memcpy(hb + o_val, vals, sizeof(float) * (size_t)nnz);
  memcpy(hb + o_lab, labels, sizeof(int32_t) * (size_t)nlab);
  // The input copy runs on a stream of its own, beside the kernels of the previous step, and the host waits for
  // it here (the device is busy with that step meanwhile).  Nothing but the step's kernels then goes into the
  // compute stream, so consecutive steps keep their kernel-to-kernel overlap; the result comes back through the
  // set's mapped record, written by the update kernel.  (The device buffer of this set was last read three steps
  // ago, by kernels that had finished before the result collected last could be written.)
  CU(cudaMemcpyAsync(db, hb, total, cudaMemcpyHostToDevice, c->st_copy_in));
  CU(cudaEventRecord(c->st_in[b], c->st_copy_in));
  CU(cudaEventSynchronize(c->st_in[b]));
  c->st_seq[b] = ++c->st_counter;
  dslide_status s = train_step_impl(ctx, batch, (const int32_t*)(db + o_rp), (const int32_t*)(db + o_col),
                                    (const float*)(db + o_val), (const int32_t*)(db + o_lp),
                                    (const int32_t*)(db + o_lab), nullptr, c->st_res_dev[b], c->st_seq[b]);
  if (s != DSLIDE_OK) { cudaStreamSynchronize(st); return s; }
  c->st_pending[b] = 1;
  return DSLIDE_OK;
}

}  // namespace

dslide_status dslide_train_step_host(dslide_ctx* ctx, int32_t batch, const int32_t* row_ptr, const int32_t* col_idx,
                                     const float* vals, const int32_t* label_ptr, const int32_t* labels,
                                     float* loss_out) {
  if (!ctx || !row_ptr || !col_idx || !vals || !label_ptr || !labels) return DSLIDE_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (batch < 1) return DSLIDE_ERR_INVALID_ARG;
  if (batch > c->cfg.max_batch) return DSLIDE_ERR_OVERFLOW;
  // results of earlier pipelined steps that nobody collected are dropped (their status stays sticky on the device)
  for (int b = 0; b < ST_SETS; ++b)
    if (c->st_pending[b]) { dslide_status w = take_result(c, b, nullptr); if (w == DSLIDE_ERR_CUDA) return w; }
  const int b = c->st_next;
  dslide_status s = enqueue_host_step(ctx, b, batch, row_ptr, col_idx, vals, label_ptr, labels);
  if (s != DSLIDE_OK) return s;
  c->st_next = (b + 1) % ST_SETS;
  s = take_result(c, b, loss_out);
  return drain_and_clear(c, s);
}

dslide_status dslide_train_step_host_async(dslide_ctx* ctx, int32_t batch, const int32_t* row_ptr,
                                           const int32_t* col_idx, const float* vals, const int32_t* label_ptr,
                                           const int32_t* labels, float* prev_loss_out, int32_t* have_prev) {
  if (!ctx || !row_ptr || !col_idx || !vals || !label_ptr || !labels) return DSLIDE_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (batch < 1) return DSLIDE_ERR_INVALID_ARG;
  if (batch > c->cfg.max_batch) return DSLIDE_ERR_OVERFLOW;
  const int b = c->st_next;
  // the set about to be reused belongs to the step three calls back, whose result was handed out long ago -- unless a
  // call in between failed: then it is dropped here and the stream is drained, so that no kernel still reads the set
  if (c->st_pending[b]) {
    dslide_status w = take_result(c, b, nullptr);
    if (w == DSLIDE_ERR_CUDA) return w;
    CU(cudaStreamSynchronize(c->stream));
  }
  dslide_status s = enqueue_host_step(ctx, b, batch, row_ptr, col_idx, vals, label_ptr, labels);
  if (s != DSLIDE_OK) return s;
  c->st_next = (b + 1) % ST_SETS;
  // while the device works on this step, collect the previous one
  const int prev = (b + ST_SETS - 1) % ST_SETS;
  const int had = c->st_pending[prev];
  if (have_prev) *have_prev = had;
  return take_result(c, prev, prev_loss_out);
}

dslide_status dslide_host_result(dslide_ctx* ctx, float* loss_out, int32_t* have) {
  if (!ctx) return DSLIDE_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  const int newest = (c->st_next + ST_SETS - 1) % ST_SETS, older = (c->st_next + ST_SETS - 2) % ST_SETS;
  dslide_status s_old = take_result(c, older, nullptr);     // only pending if its collection was skipped
  if (have) *have = c->st_pending[newest];
  dslide_status s = take_result(c, newest, loss_out);
  return drain_and_clear(c, s != DSLIDE_OK ? s : s_old);
}

dslide_status dslide_predict_topk(dslide_ctx* ctx, int32_t batch, const int32_t* row_ptr, const int32_t* col_idx,
                                  const float* vals, int32_t k, int32_t dense, int32_t* out_ids, float* out_scores) {
  if (!ctx || !row_ptr || !col_idx || !vals || !out_ids || !out_scores) return DSLIDE_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (batch < 1 || k < 1 || k > 64) return DSLIDE_ERR_INVALID_ARG;
  if (batch > c->cfg.max_batch) return DSLIDE_ERR_OVERFLOW;
  CU(launch_predict(c, batch, row_ptr, col_idx, vals, k, (dense || c->dense) ? 1 : 0, out_ids, out_scores));
  return DSLIDE_OK;
}

dslide_status dslide_sync(dslide_ctx* ctx) {
  if (!ctx) return DSLIDE_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  int status = 0;
  CU(cudaMemcpyAsync(&status, &c->dstate->status, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  CU(cudaStreamSynchronize(c->stream));
  if (status != 0) {
    CU(cudaMemsetAsync(&c->dstate->status, 0, sizeof(int), c->stream));
    CU(cudaStreamSynchronize(c->stream));
  }
  return (dslide_status)status;
}

dslide_status dslide_tensor_info(dslide_ctx* ctx, int32_t which, int64_t* nbytes, int32_t* dtype) {
  if (!ctx || !nbytes) return DSLIDE_ERR_INVALID_ARG;
  TensorRef t = tensor_ref(&ctx->c, which);
  if (t.bytes < 0) return DSLIDE_ERR_INVALID_ARG;
  if (ctx->c.dense && (which == DSLIDE_T_BUCKET_OFF || which == DSLIDE_T_BUCKET_IDS)) t.bytes = 0;
  *nbytes = t.bytes;
  if (dtype)
    *dtype = which == DSLIDE_T_COUNTERS ? DSLIDE_DT_I64
             : which == DSLIDE_T_PROJ1 ? DSLIDE_DT_I8
             : ((which >= DSLIDE_T_HASH_IDX && which <= DSLIDE_T_BUCKET_IDS) || which == DSLIDE_T_BUCKET1_OFF ||
                which == DSLIDE_T_BUCKET1_IDS) ? DSLIDE_DT_I32 : DSLIDE_DT_F32;
  return DSLIDE_OK;
}

dslide_status dslide_get_tensor(dslide_ctx* ctx, int32_t which, void* host_dst, int64_t nbytes) {
  if (!ctx || !host_dst) return DSLIDE_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  int64_t want = 0;
  dslide_status s = dslide_tensor_info(ctx, which, &want, nullptr);
  if (s != DSLIDE_OK) return s;
  if (nbytes != want) return DSLIDE_ERR_INVALID_ARG;
  if (which == DSLIDE_T_COUNTERS) {
    int64_t v[3] = {c->t_host, c->r_host, c->next_rebuild};
    memcpy(host_dst, v, sizeof(v));
    return DSLIDE_OK;
  }
  if (want == 0) return DSLIDE_OK;
  if (which == DSLIDE_T_BUCKET_IDS && c->place_path && c->ids_ordered_above > 1) {
    // the step only needs buckets beyond the cap in order; a reader gets every bucket ascending
    CU(launch_order_buckets(c, 1));
    c->ids_ordered_above = 1;
  }
  const TensorRef tr = tensor_ref(c, which);
  if (tr.pitch) CU(cudaMemcpy2DAsync(host_dst, sizeof(float), tr.ptr, (size_t)tr.pitch, sizeof(float), (size_t)want / sizeof(float),
                                     cudaMemcpyDeviceToHost, c->stream));
  else CU(cudaMemcpyAsync(host_dst, tr.ptr, (size_t)want, cudaMemcpyDeviceToHost, c->stream));
  return drain(c);
}

dslide_status dslide_set_tensor(dslide_ctx* ctx, int32_t which, const void* host_src, int64_t nbytes) {
  if (!ctx || !host_src) return DSLIDE_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  int64_t want = 0;
  dslide_status s = dslide_tensor_info(ctx, which, &want, nullptr);
  if (s != DSLIDE_OK) return s;
  if (nbytes != want) return DSLIDE_ERR_INVALID_ARG;
  if (which == DSLIDE_T_COUNTERS) {
    int64_t v[3];
    memcpy(v, host_src, sizeof(v));
    if (v[0] < 0 || v[1] < 0) return DSLIDE_ERR_INVALID_ARG;
    c->t_host = v[0]; c->r_host = v[1]; c->next_rebuild = v[2];
    // the device-side slots are indexed by the step's parity: make the slot of the next step the clean one
    CU(cudaMemsetAsync(c->dstate->n_own, 0, sizeof(c->dstate->n_own), c->stream));
    CU(cudaMemsetAsync(c->dstate->n_hot, 0, sizeof(c->dstate->n_hot), c->stream));
    CU(cudaMemsetAsync(c->dstate->n_med, 0, sizeof(c->dstate->n_med), c->stream));
    CU(cudaMemsetAsync(c->dstate->ticket, 0, sizeof(c->dstate->ticket), c->stream));
    CU(cudaMemsetAsync(c->dstate->acc, 0, sizeof(c->dstate->acc), c->stream));
    return drain(c);
  }
  if (which == DSLIDE_T_HASH_IDX) {
    const int32_t* ix = (const int32_t*)host_src;
    for (int64_t i = 0; i < want / 4; ++i)
      if (ix[i] < 0 || ix[i] >= c->H) return DSLIDE_ERR_INVALID_ARG;
  }
  if (which == DSLIDE_T_BUCKET_OFF || which == DSLIDE_T_BUCKET_IDS || which == DSLIDE_T_BUCKET1_OFF ||
      which == DSLIDE_T_BUCKET1_IDS) return DSLIDE_ERR_INVALID_ARG;  // derived state
  if (which == DSLIDE_T_PROJ1) {
    const signed char* e = (const signed char*)host_src;
    for (int64_t i = 0; i < want; ++i)
      if (e[i] < -1 || e[i] > 1) return DSLIDE_ERR_INVALID_ARG;
  }
  if (want == 0) return DSLIDE_OK;
  const TensorRef tr = tensor_ref(c, which);
  if (tr.pitch) CU(cudaMemcpy2DAsync(tr.ptr, (size_t)tr.pitch, host_src, sizeof(float), sizeof(float), (size_t)want / sizeof(float),
                                     cudaMemcpyHostToDevice, c->stream));
  else CU(cudaMemcpyAsync(tr.ptr, host_src, (size_t)want, cudaMemcpyHostToDevice, c->stream));
  return drain(c);
}

dslide_status dslide_last_info(dslide_ctx* ctx, int32_t which, int64_t* nbytes, int32_t* stride) {
  if (!ctx || !nbytes) return DSLIDE_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  const int64_t B = c->cfg.max_batch, S = c->act_stride;
  if (stride) *stride = c->act_stride;
  switch (which) {
    case DSLIDE_LAST_HIDDEN: case DSLIDE_LAST_DHIDDEN: *nbytes = B * c->H * 4; return DSLIDE_OK;
    case DSLIDE_LAST_CODES: *nbytes = B * c->L * 4; return DSLIDE_OK;
    case DSLIDE_LAST_ACT_COUNT: case DSLIDE_LAST_LOSS: *nbytes = B * 4; return DSLIDE_OK;
    case DSLIDE_LAST_ACT_IDS: *nbytes = c->dense ? 0 : B * S * 4; return DSLIDE_OK;
    case DSLIDE_LAST_ACT_LOGIT: case DSLIDE_LAST_ACT_PROB: case DSLIDE_LAST_ACT_ERR: *nbytes = B * S * 4; return DSLIDE_OK;
    case DSLIDE_LAST_CODES1: *nbytes = B * c->L1 * 4; return DSLIDE_OK;
    case DSLIDE_LAST_HIDDEN_MASK: *nbytes = c->L1 > 0 ? B * c->Hw * 4 : 0; return DSLIDE_OK;
  }
  return DSLIDE_ERR_INVALID_ARG;
}

dslide_status dslide_get_last(dslide_ctx* ctx, int32_t which, void* host_dst, int64_t nbytes) {
  if (!ctx || !host_dst || nbytes < 0) return DSLIDE_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  int64_t size = 0;
  dslide_status s = dslide_last_info(ctx, which, &size, nullptr);
  if (s != DSLIDE_OK) return s;
  const void* src = nullptr;
  switch (which) {
    case DSLIDE_LAST_HIDDEN: src = c->h; break;
    case DSLIDE_LAST_DHIDDEN: src = c->dh; break;
    case DSLIDE_LAST_CODES: src = c->codes; break;
    case DSLIDE_LAST_ACT_COUNT: src = c->act_cnt; break;
    case DSLIDE_LAST_LOSS: src = c->loss; break;
    case DSLIDE_LAST_ACT_IDS: src = c->act_ids; break;
    case DSLIDE_LAST_ACT_LOGIT: src = c->act_z; break;
    case DSLIDE_LAST_ACT_PROB: src = c->act_p; break;
    case DSLIDE_LAST_ACT_ERR: src = c->act_g; break;
    case DSLIDE_LAST_CODES1: src = c->codes1; break;
    case DSLIDE_LAST_HIDDEN_MASK: src = c->hmask; break;
  }
  int64_t n = nbytes < size ? nbytes : size;
  if (n == 0 || !src) return DSLIDE_OK;
  CU(cudaMemcpyAsync(host_dst, src, (size_t)n, cudaMemcpyDeviceToHost, c->stream));
  return drain(c);
}

dslide_status dslide_last_stats(dslide_ctx* ctx, int64_t out[4]) {
  if (!ctx || !out) return DSLIDE_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  DevState s;
  CU(cudaMemcpyAsync(&s, c->dstate, sizeof(s), cudaMemcpyDeviceToHost, c->stream));
  CU(cudaStreamSynchronize(c->stream));
  const int q = (int)((c->t_host + 1) & 1);      // parity of the last finished step
  out[0] = (int64_t)s.last[0]; out[1] = c->dense ? c->N : (int64_t)s.n_own[q][0]; out[2] = (int64_t)s.n_own[q][1];
  out[3] = (int64_t)s.last[1];
  static_assert((int)KID_COUNT == (int)DSLIDE_K_COUNT, "kernel id enums out of step");
  return DSLIDE_OK;
}

dslide_status dslide_cum_stats(dslide_ctx* ctx, int64_t out[6], int32_t reset) {
  if (!ctx || !out) return DSLIDE_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  DevState s;
  CU(cudaMemcpyAsync(&s, c->dstate, sizeof(s), cudaMemcpyDeviceToHost, c->stream));
  CU(cudaStreamSynchronize(c->stream));
  for (int i = 0; i < 6; ++i) out[i] = (int64_t)s.cum[i];
  if (reset) {
    CU(cudaMemsetAsync(c->dstate->cum, 0, sizeof(s.cum), c->stream));
    CU(cudaStreamSynchronize(c->stream));
  }
  return DSLIDE_OK;
}

dslide_status dslide_profile_begin(dslide_ctx* ctx) {
  if (!ctx) return DSLIDE_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (c->profiling) return DSLIDE_ERR_STATE;
  if (!c->prof) c->prof = new (std::nothrow) std::vector<ProfRec>();
  if (!c->prof) return DSLIDE_ERR_OOM;
  static_cast<std::vector<ProfRec>*>(c->prof)->reserve(1 << 16);
  c->profiling = 1;
  return DSLIDE_OK;
}

dslide_status dslide_profile_end(dslide_ctx* ctx, double ms[DSLIDE_K_COUNT], int64_t launches[DSLIDE_K_COUNT]) {
  if (!ctx || !ms || !launches) return DSLIDE_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (!c->profiling) return DSLIDE_ERR_STATE;
  c->profiling = 0;
  CU(cudaStreamSynchronize(c->stream));
  for (int i = 0; i < DSLIDE_K_COUNT; ++i) { ms[i] = 0.0; launches[i] = 0; }
  auto* v = static_cast<std::vector<ProfRec>*>(c->prof);
  for (auto& r : *v) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, r.beg, r.end) == cudaSuccess && r.kid >= 0 && r.kid < DSLIDE_K_COUNT) {
      ms[r.kid] += t;
      launches[r.kid] += 1;
    }
    cudaEventDestroy(r.beg);
    cudaEventDestroy(r.end);
  }
  v->clear();
  return DSLIDE_OK;
}

int64_t dslide_kernel_launches(const dslide_ctx* ctx) { return ctx ? ctx->c.launches : 0; }

}  // extern "C"
