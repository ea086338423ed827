"""Thin ctypes binding over the C ABI in include/dslide.h.

Argument marshalling only: every step of the training path runs in the CUDA
kernels of libdslide.so.  torch is used for device memory and streams.  The
functions carry the names of the C entry points.  Importing this module fails
loudly when the library has not been built (python -m paper_2201_12667_b200.build)
-- there is no CPU fallback.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdslide.so")

if not os.path.exists(LIB_PATH):
    raise ImportError("libdslide.so is missing: build it with `python -m paper_2201_12667_b200.build` "
                      "(needs nvcc); there is no fallback path")
_lib = C.CDLL(LIB_PATH)

OK, ERR_INVALID_ARG, ERR_OOM, ERR_CUDA, ERR_OVERFLOW, ERR_BAD_INDEX, ERR_STATE, ERR_TIMEOUT = range(8)
SIMHASH, DWTA = 0, 1

T_NAMES = ["W1", "b1", "W2", "b2", "mW1", "vW1", "mb1", "vb1", "mW2", "vW2", "mb2", "vb2",
           "hash_idx", "hash_sign", "bucket_off", "bucket_ids", "counters", "proj1", "bucket1_off", "bucket1_ids"]
T = {n: i for i, n in enumerate(T_NAMES)}
_T_DTYPE = {"hash_idx": np.int32, "hash_sign": np.int32, "bucket_off": np.int32, "bucket_ids": np.int32,
            "counters": np.int64, "proj1": np.int8, "bucket1_off": np.int32, "bucket1_ids": np.int32}
LAST_NAMES = ["hidden", "codes", "act_count", "act_ids", "act_logit", "act_prob", "act_err", "loss", "dhidden",
              "codes1", "hidden_mask"]
LAST = {n: i for i, n in enumerate(LAST_NAMES)}
_LAST_DTYPE = {"codes": np.uint32, "act_count": np.int32, "act_ids": np.int32, "codes1": np.uint32, "hidden_mask": np.uint32}


class Config(C.Structure):
    _fields_ = [
        ("input_dim", C.c_int32), ("hidden_dim", C.c_int32), ("output_dim", C.c_int32),
        ("hash_family", C.c_int32), ("K", C.c_int32), ("L", C.c_int32),
        ("dwta_bin_size", C.c_int32), ("srp_nnz", C.c_int32), ("bucket_cap", C.c_int32),
        ("rebuild_period0", C.c_int32), ("rebuild_growth_lambda", C.c_float),
        ("redraw_hash_fns", C.c_int32), ("force_dense", C.c_int32),
        ("max_batch", C.c_int32), ("max_labels", C.c_int32), ("max_active_per_sample", C.c_int32),
        ("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
        ("init_std", C.c_float), ("seed", C.c_uint64), ("device", C.c_int32), ("dedup_mode", C.c_int32),
        ("stream", C.c_void_p), ("dwta_densify", C.c_int32), ("sample_budget", C.c_int32), ("budget_fill", C.c_int32),
        ("inputs_ready", C.c_int32), ("hidden_K", C.c_int32), ("hidden_L", C.c_int32), ("hidden_cap", C.c_int32),
    ]


_vp, _i32, _i64 = C.c_void_p, C.c_int32, C.c_int64
_SIGS = {
    "dslide_init": (_i32, [C.POINTER(Config), C.POINTER(_vp)]),
    "dslide_destroy": (_i32, [_vp]),
    "dslide_rebuild_tables": (_i32, [_vp]),
    "dslide_build_tables": (_i32, [_vp]),
    "dslide_train_step": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _vp, _vp]),
    "dslide_train_step_host": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _vp, C.POINTER(C.c_float)]),
    "dslide_train_step_host_async": (_i32, [_vp, _i32, _vp, _vp, _vp, _vp, _vp, C.POINTER(C.c_float), C.POINTER(_i32)]),
    "dslide_host_result": (_i32, [_vp, C.POINTER(C.c_float), C.POINTER(_i32)]),
    "dslide_predict_topk": (_i32, [_vp, _i32, _vp, _vp, _vp, _i32, _i32, _vp, _vp]),
    "dslide_sync": (_i32, [_vp]),
    "dslide_tensor_info": (_i32, [_vp, _i32, C.POINTER(_i64), C.POINTER(_i32)]),
    "dslide_get_tensor": (_i32, [_vp, _i32, _vp, _i64]),
    "dslide_set_tensor": (_i32, [_vp, _i32, _vp, _i64]),
    "dslide_last_info": (_i32, [_vp, _i32, C.POINTER(_i64), C.POINTER(_i32)]),
    "dslide_get_last": (_i32, [_vp, _i32, _vp, _i64]),
    "dslide_last_stats": (_i32, [_vp, C.POINTER(_i64)]),
    "dslide_cum_stats": (_i32, [_vp, C.POINTER(_i64), _i32]),
    "dslide_profile_begin": (_i32, [_vp]),
    "dslide_profile_end": (_i32, [_vp, C.POINTER(C.c_double), C.POINTER(_i64)]),
    "dslide_bucket_sort_static": (_i32, [_vp, _i32, _i32, _vp, _vp, _vp]),
    "dslide_kernel_launches": (_i64, [_vp]),
    "dslide_status_str": (C.c_char_p, [_i32]),
}
EXPORTS = sorted(_SIGS)
for _name, (_res, _args) in _SIGS.items():
    _f = getattr(_lib, _name)
    _f.restype = _res
    _f.argtypes = _args


class DslideError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__("%s: %s (%d)" % (where, _lib.dslide_status_str(status).decode(), status))


def _check(status, where):
    if status != OK:
        raise DslideError(status, where)


def _dptr(t):
    """Device pointer of a contiguous CUDA tensor (or None)."""
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous()
    return t.data_ptr()


def make_config(*, input_dim, hidden_dim, output_dim, hash_family=DWTA, K=6, L=50, dwta_bin_size=8, srp_nnz=0,
                bucket_cap=128, rebuild_period0=50, rebuild_growth_lambda=0.0, redraw_hash_fns=1, force_dense=0,
                max_batch=256, max_labels=16, max_active_per_sample=0, lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8,
                init_std=0.01, seed=0, device=0, dedup_mode=0, stream=None, dwta_densify=0, sample_budget=0, budget_fill=0,
                inputs_ready=0, hidden_K=0, hidden_L=0, hidden_cap=0):
    if stream is None:
        import torch
        stream = torch.cuda.current_stream(device).cuda_stream
    return Config(input_dim, hidden_dim, output_dim, hash_family, K, L, dwta_bin_size, srp_nnz, bucket_cap,
                  rebuild_period0, rebuild_growth_lambda, redraw_hash_fns, force_dense, max_batch, max_labels,
                  max_active_per_sample, lr, beta1, beta2, eps, init_std, seed, device, dedup_mode, stream, dwta_densify, sample_budget, budget_fill,
                  inputs_ready, hidden_K, hidden_L, hidden_cap)


# ---- the C entry points, same names ---------------------------------------------------------
def dslide_init(cfg):
    ctx = _vp()
    _check(_lib.dslide_init(C.byref(cfg), C.byref(ctx)), "dslide_init")
    return ctx


def dslide_destroy(ctx):
    _check(_lib.dslide_destroy(ctx), "dslide_destroy")


def dslide_rebuild_tables(ctx):
    _check(_lib.dslide_rebuild_tables(ctx), "dslide_rebuild_tables")


def dslide_build_tables(ctx):
    _check(_lib.dslide_build_tables(ctx), "dslide_build_tables")


def dslide_train_step(ctx, batch, row_ptr, col_idx, vals, label_ptr, labels, loss_out=None):
    """All array arguments are CUDA tensors (int32 / float32); loss_out a 1-element CUDA float tensor or None."""
    _check(_lib.dslide_train_step(ctx, batch, _dptr(row_ptr), _dptr(col_idx), _dptr(vals), _dptr(label_ptr),
                                  _dptr(labels), _dptr(loss_out)), "dslide_train_step")


def dslide_train_step_host(ctx, batch, row_ptr, col_idx, vals, label_ptr, labels):
    """Array arguments are HOST tensors or numpy arrays (int32 / float32).  Returns the mean loss."""
    loss = C.c_float(0.0)
    ptr = [a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data for a in (row_ptr, col_idx, vals, label_ptr, labels)]
    _check(_lib.dslide_train_step_host(ctx, batch, *ptr, C.byref(loss)), "dslide_train_step_host")
    return loss.value


def dslide_train_step_host_async(ctx, batch, row_ptr, col_idx, vals, label_ptr, labels):
    """Pipelined host-buffer step: enqueues this batch, returns the mean loss of the PREVIOUS such step (None if none)."""
    loss, have = C.c_float(0.0), _i32(0)
    ptr = [a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data for a in (row_ptr, col_idx, vals, label_ptr, labels)]
    _check(_lib.dslide_train_step_host_async(ctx, batch, *ptr, C.byref(loss), C.byref(have)), "dslide_train_step_host_async")
    return loss.value if have.value else None


def dslide_host_result(ctx):
    """Waits for the newest pipelined host-buffer step; returns its mean loss (None if none is outstanding)."""
    loss, have = C.c_float(0.0), _i32(0)
    _check(_lib.dslide_host_result(ctx, C.byref(loss), C.byref(have)), "dslide_host_result")
    return loss.value if have.value else None


def dslide_predict_topk(ctx, batch, row_ptr, col_idx, vals, k, dense, out_ids, out_scores):
    _check(_lib.dslide_predict_topk(ctx, batch, _dptr(row_ptr), _dptr(col_idx), _dptr(vals), k, int(dense),
                                    _dptr(out_ids), _dptr(out_scores)), "dslide_predict_topk")


def dslide_sync(ctx, check=True):
    s = _lib.dslide_sync(ctx)
    if check:
        _check(s, "dslide_sync")
    return s


_DT = [np.float32, np.int32, np.int64, np.int8]       # DSLIDE_DT_*


def dslide_get_tensor(ctx, name):
    n, code = _i64(), _i32()
    _check(_lib.dslide_tensor_info(ctx, T[name], C.byref(n), C.byref(code)), "dslide_tensor_info")
    dt = np.dtype(_DT[code.value])
    out = np.empty(n.value // dt.itemsize, dtype=dt)
    if n.value:
        _check(_lib.dslide_get_tensor(ctx, T[name], out.ctypes.data, n.value), "dslide_get_tensor")
    return out


def dslide_set_tensor(ctx, name, arr):
    dt = np.dtype(_T_DTYPE.get(name, np.float32))
    a = np.ascontiguousarray(np.asarray(arr).reshape(-1), dtype=dt)
    _check(_lib.dslide_set_tensor(ctx, T[name], a.ctypes.data, a.nbytes), "dslide_set_tensor")


def dslide_get_last(ctx, name, batch):
    """Snapshot array `name` of the last training step for the first `batch` samples."""
    n, stride = _i64(), _i32()
    _check(_lib.dslide_last_info(ctx, LAST[name], C.byref(n), C.byref(stride)), "dslide_last_info")
    dt = np.dtype(_LAST_DTYPE.get(name, np.float32))
    total = n.value // dt.itemsize
    if total == 0:
        return np.zeros((batch, 0), dtype=dt)
    per = total // _max_batch_of(ctx)
    out = np.empty(batch * per, dtype=dt)
    _check(_lib.dslide_get_last(ctx, LAST[name], out.ctypes.data, out.nbytes), "dslide_get_last")
    return out.reshape(batch, per) if per > 1 else out


def _max_batch_of(ctx):
    # rows of the snapshot array = max_batch; recover it from the loss array, which has one float per sample
    n = _i64()
    _check(_lib.dslide_last_info(ctx, LAST["loss"], C.byref(n), None), "dslide_last_info")
    return n.value // 4


def dslide_last_stats(ctx):
    out = (_i64 * 4)()
    _check(_lib.dslide_last_stats(ctx, out), "dslide_last_stats")
    return dict(sum_active=out[0], touched_w2=out[1], touched_w1=out[2], nnz=out[3])


KERNEL_NAMES = ["forward", "adam_dense", "adam", "draw_hash", "hash_neurons", "bucket_scan", "sort_hist", "sort_scan",
                "sort_scatter", "predict", "init", "place_ids", "order_buckets"]


def dslide_cum_stats(ctx, reset=False):
    out = (_i64 * 6)()
    _check(_lib.dslide_cum_stats(ctx, out, int(reset)), "dslide_cum_stats")
    return dict(steps=out[0], sum_active=out[1], touched_w2=out[2], touched_w1=out[3], nnz=out[4], fetched=out[5])


def dslide_profile_begin(ctx):
    _check(_lib.dslide_profile_begin(ctx), "dslide_profile_begin")


def dslide_profile_end(ctx):
    """-> {kernel name: (milliseconds, launches)} for the kernels launched since dslide_profile_begin."""
    n = len(KERNEL_NAMES)
    ms, cnt = (C.c_double * n)(), (_i64 * n)()
    _check(_lib.dslide_profile_end(ctx, ms, cnt), "dslide_profile_end")
    return {KERNEL_NAMES[i]: (ms[i], cnt[i]) for i in range(n) if cnt[i]}


STATIC_SORT_MAX_N = 262144
STATIC_SORT_MAX_BITS = 18


def dslide_bucket_sort_static(codes, n, bits, bucket_off, bucket_ids, stream=None):
    """Group ids 0..n-1 by bucket code without allocating (see include/dslide.h).

    codes: CUDA uint32/int32 tensor [n]; bucket_off: CUDA int32 tensor [2**bits + 1]; bucket_ids: CUDA int32
    tensor [n]; stream: a torch stream or None for torch's current stream.  The library allocates nothing;
    the tensors are the caller's.
    """
    import torch
    st = (stream or torch.cuda.current_stream()).cuda_stream
    _check(_lib.dslide_bucket_sort_static(_dptr(codes), n, bits, _dptr(bucket_off), _dptr(bucket_ids), st),
           "dslide_bucket_sort_static")


def dslide_kernel_launches(ctx):
    return int(_lib.dslide_kernel_launches(ctx))
