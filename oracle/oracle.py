"""ctypes harness around oracle/slide_oracle.c -- TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may
import this module.  It builds the C oracle twice (REAL=float, the parity
target, and REAL=double, used by the gradient and dense-limit pins) and
exposes its state as numpy views.  It shares nothing with the CUDA library.
"""
import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "slide_oracle.c")

# -ffp-contract=off: a*b+c is never fused behind the code's back; the fused
# multiply-adds the definition asks for are explicit fmaf/fma calls.
_CFLAGS = ["-O2", "-ffp-contract=off", "-fPIC", "-shared", "-std=c99", "-fno-fast-math"]


def lib_path(real):
    return os.path.join(_HERE, "libslide_oracle_%s.so" % {"float": "f32", "double": "f64", "float_omp": "f32_omp"}[real])


def build(force=False):
    """Compile the variants of the oracle with gcc (a few seconds): fp32, fp64, and fp32 with OpenMP (the same
    source; only used to time the oracle on all host cores, and pinned bit-identical to the plain fp32 build)."""
    for real in ("float", "double", "float_omp"):
        out = lib_path(real)
        if (not force and os.path.exists(out)
                and os.path.getmtime(out) >= os.path.getmtime(_SRC)):
            continue
        tmp = out + ".tmp%d" % os.getpid()
        extra = ["-fopenmp"] if real.endswith("_omp") else []
        subprocess.check_call(["gcc"] + _CFLAGS + extra + ["-DREAL=%s" % real.split("_")[0], _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, out)


class OrcConfig(C.Structure):
    _fields_ = [
        ("D", C.c_int32), ("H", C.c_int32), ("N", C.c_int32),
        ("family", C.c_int32), ("K", C.c_int32), ("L", C.c_int32),
        ("bin_size", C.c_int32), ("srp_nnz", C.c_int32), ("bucket_cap", C.c_int32),
        ("rebuild_period0", C.c_int32), ("redraw", C.c_int32), ("force_dense", C.c_int32),
        ("max_active", C.c_int32), ("densify", C.c_int32), ("budget", C.c_int32), ("budget_fill", C.c_int32),
        ("rebuild_lambda", C.c_double),
        ("lr", C.c_double), ("beta1", C.c_double), ("beta2", C.c_double), ("eps", C.c_double),
        ("init_std", C.c_double),
        ("seed", C.c_uint64),
        ("hidden_K", C.c_int32), ("hidden_L", C.c_int32), ("hidden_cap", C.c_int32),
    ]


# must match the enum in slide_oracle.c
NAMES = ["W1", "b1", "W2", "b2", "mW1", "vW1", "mb1", "vb1", "mW2", "vW2", "mb2", "vb2",
         "dW1", "db1", "dW2", "db2", "hash_idx", "hash_sign", "bucket_off", "bucket_ids",
         "h", "dh", "codes", "act_ptr", "act_ids", "act_z", "act_p", "act_g", "loss",
         "proj1", "bucket1_off", "bucket1_ids", "codes1", "hact"]
_WHICH = {n: i for i, n in enumerate(NAMES)}
_INT_TYPES = {"hash_idx": np.int32, "hash_sign": np.int32, "bucket_off": np.int32, "bucket_ids": np.int32,
              "codes": np.uint32, "act_ptr": np.int64, "act_ids": np.int32,
              "proj1": np.int8, "bucket1_off": np.int32, "bucket1_ids": np.int32, "codes1": np.uint32, "hact": np.uint8}

SIMHASH, DWTA = 0, 1

_libs = {}


def _load(real):
    if real not in _libs:
        build()
        lib = C.CDLL(lib_path(real))
        lib.orc_create.restype = C.c_void_p
        lib.orc_create.argtypes = [C.POINTER(OrcConfig)]
        lib.orc_destroy.argtypes = [C.c_void_p]
        lib.orc_ptr.restype = C.c_void_p
        lib.orc_ptr.argtypes = [C.c_void_p, C.c_int32]
        lib.orc_count.restype = C.c_int64
        lib.orc_count.argtypes = [C.c_void_p, C.c_int32]
        for f in ("orc_step_count", "orc_rebuild_count", "orc_next_rebuild"):
            getattr(lib, f).restype = C.c_int64
            getattr(lib, f).argtypes = [C.c_void_p]
        lib.orc_set_counters.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64]
        for f in ("orc_bits", "orc_idx_per_fn", "orc_last_error"):
            getattr(lib, f).restype = C.c_int32
            getattr(lib, f).argtypes = [C.c_void_p]
        lib.orc_rng.restype = C.c_uint64
        lib.orc_rng.argtypes = [C.c_uint64] * 4
        lib.orc_threads.restype = C.c_int32
        lib.orc_threads.argtypes = []
        lib.orc_mix64.restype = C.c_uint64
        lib.orc_mix64.argtypes = [C.c_uint64]
        lib.orc_draw_hash.argtypes = [C.c_void_p, C.c_int64]
        lib.orc_build_tables.argtypes = [C.c_void_p]
        lib.orc_build_tables1.argtypes = [C.c_void_p]
        lib.orc_draw_hash1.argtypes = [C.c_void_p, C.c_int64]
        lib.orc_rebuild_tables.argtypes = [C.c_void_p]
        lib.orc_hash_vec.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        lib.orc_hash_query.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        lib.orc_forward.restype = C.c_int32
        lib.orc_forward.argtypes = [C.c_void_p, C.c_int32] + [C.c_void_p] * 5
        lib.orc_backward.argtypes = [C.c_void_p]
        lib.orc_adam.argtypes = [C.c_void_p]
        lib.orc_schedule.restype = C.c_int32
        lib.orc_schedule.argtypes = [C.c_void_p]
        lib.orc_train_step.restype = C.c_int32
        lib.orc_train_step.argtypes = [C.c_void_p, C.c_int32] + [C.c_void_p] * 5 + [C.POINTER(C.c_double)]
        lib.orc_predict_topk.restype = C.c_int32
        lib.orc_predict_topk.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        _libs[real] = lib
    return _libs[real]


def rng(seed, stream, r, ctr):
    return int(_load("float").orc_rng(seed, stream, r, ctr))


def mix64(z):
    """The generator's output function alone (pinned against the published splitmix64 outputs)."""
    return int(_load("float").orc_mix64(z))


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


class Oracle:
    """One model instance of the CPU oracle.  `real` is "float", "double" or "float_omp" (fp32 on all cores)."""

    def __init__(self, real="float", **kw):
        self.real = real
        self.dtype = np.float64 if real == "double" else np.float32
        self.lib = _load(real)
        d = dict(family=SIMHASH, bin_size=8, srp_nnz=0, bucket_cap=128, rebuild_period0=0, redraw=1,
                 force_dense=0, max_active=0, densify=0, budget=0, budget_fill=0, rebuild_lambda=0.0, lr=1e-4, beta1=0.9, beta2=0.999,
                 eps=1e-8, init_std=0.01, seed=0, hidden_K=0, hidden_L=0, hidden_cap=0)
        d.update(kw)
        self.cfg = OrcConfig(**d)
        self.o = self.lib.orc_create(C.byref(self.cfg))
        if not self.o:
            raise MemoryError("orc_create failed")
        self.H, self.N, self.D, self.L, self.K = d["H"], d["N"], d["D"], d["L"], d["K"]

    @property
    def threads(self):
        """Worker threads the library uses (1 unless it is the OpenMP build)."""
        return int(self.lib.orc_threads())

    def close(self):
        if self.o:
            self.lib.orc_destroy(self.o)
            self.o = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- state ---------------------------------------------------------
    def view(self, name):
        """A numpy view (no copy) of one array of the oracle; valid until the next call that reallocates it."""
        w = _WHICH[name]
        n = self.lib.orc_count(self.o, w)
        dt = _INT_TYPES.get(name, self.dtype)
        if n <= 0:
            return np.zeros(0, dtype=dt)
        ptr = self.lib.orc_ptr(self.o, w)
        buf = (C.c_char * (n * np.dtype(dt).itemsize)).from_address(ptr)
        return np.frombuffer(buf, dtype=dt, count=n)

    def get(self, name):
        return self.view(name).copy()

    def set(self, name, arr):
        v = self.view(name)
        v[...] = np.asarray(arr, dtype=v.dtype).reshape(-1)

    @property
    def t(self):
        return self.lib.orc_step_count(self.o)

    @property
    def r(self):
        return self.lib.orc_rebuild_count(self.o)

    @property
    def next_rebuild(self):
        return self.lib.orc_next_rebuild(self.o)

    def set_counters(self, t, r, next_rebuild):
        self.lib.orc_set_counters(self.o, t, r, next_rebuild)

    @property
    def bits(self):
        return self.lib.orc_bits(self.o)

    @property
    def idx_per_fn(self):
        return self.lib.orc_idx_per_fn(self.o)

    # -- the algorithm -------------------------------------------------
    def draw_hash(self, r):
        self.lib.orc_draw_hash(self.o, r)

    def build_tables(self):
        self.lib.orc_build_tables(self.o)

    def build_tables1(self):
        """Tables over the hidden neurons (LSH-sampled hidden layer)."""
        self.lib.orc_build_tables1(self.o)

    def draw_hash1(self, r):
        self.lib.orc_draw_hash1(self.o, r)

    def rebuild_tables(self):
        self.lib.orc_rebuild_tables(self.o)

    def hash_vec(self, v):
        v = np.ascontiguousarray(v, dtype=self.dtype)
        assert v.shape == (self.H,)
        out = np.zeros(self.L, dtype=np.uint32)
        self.lib.orc_hash_vec(self.o, _p(v), _p(out))
        return out

    def hash_query(self, v):
        """Codes of a query (a hidden activation): as hash_vec, plus densification of all-zero DWTA bins when set."""
        v = np.ascontiguousarray(v, dtype=self.dtype)
        assert v.shape == (self.H,)
        out = np.zeros(self.L, dtype=np.uint32)
        self.lib.orc_hash_query(self.o, _p(v), _p(out))
        return out

    def _batch(self, row_ptr, col_idx, vals, label_ptr=None, labels=None):
        row_ptr = np.ascontiguousarray(row_ptr, dtype=np.int32)
        col_idx = np.ascontiguousarray(col_idx, dtype=np.int32)
        vals = np.ascontiguousarray(vals, dtype=self.dtype)
        if label_ptr is not None:
            label_ptr = np.ascontiguousarray(label_ptr, dtype=np.int32)
            labels = np.ascontiguousarray(labels, dtype=np.int32)
        return row_ptr, col_idx, vals, label_ptr, labels

    def forward(self, row_ptr, col_idx, vals, label_ptr=None, labels=None):
        a = self._batch(row_ptr, col_idx, vals, label_ptr, labels)
        e = self.lib.orc_forward(self.o, len(a[0]) - 1, *[_p(x) for x in a])
        if e:
            raise RuntimeError("oracle forward error %d" % e)

    def backward(self):
        self.lib.orc_backward(self.o)

    def adam(self):
        self.lib.orc_adam(self.o)

    def schedule(self):
        return bool(self.lib.orc_schedule(self.o))

    def train_step(self, row_ptr, col_idx, vals, label_ptr, labels):
        a = self._batch(row_ptr, col_idx, vals, label_ptr, labels)
        loss = C.c_double(0.0)
        e = self.lib.orc_train_step(self.o, len(a[0]) - 1, *[_p(x) for x in a], C.byref(loss))
        if e:
            raise RuntimeError("oracle train_step error %d" % e)
        return loss.value

    def predict_topk(self, row_ptr, col_idx, vals, k, dense=False):
        a = self._batch(row_ptr, col_idx, vals)
        B = len(a[0]) - 1
        ids = np.zeros((B, k), dtype=np.int32)
        sc = np.zeros((B, k), dtype=self.dtype)
        e = self.lib.orc_predict_topk(self.o, B, _p(a[0]), _p(a[1]), _p(a[2]), k, int(dense), _p(ids), _p(sc))
        if e:
            raise RuntimeError("oracle predict error %d" % e)
        return ids, sc

    def active_sets(self):
        ptr = self.get("act_ptr")
        ids = self.get("act_ids")
        return [ids[ptr[s]:ptr[s + 1]] for s in range(len(ptr) - 1)]


if __name__ == "__main__":
    build(force=True)
    print("built", lib_path("float"), lib_path("double"))
