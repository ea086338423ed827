"""dslide_bucket_sort_static: the table sort for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is not theirs to call (they are handed buffers by a
host application, or have promised a fixed footprint).  The entry point under test keeps its work
space in a static device array inside the library, so the check here is simple: through the C ABI,
with buffers the test owns, it must reproduce bit for bit the tables that the ordinary entry points
(dslide_init / dslide_build_tables, read back with dslide_get_tensor) build for the same codes --
twice in a row, because every call reuses the same static array and must not see the previous call's
leftovers.  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2201_12667_b200 import binding as ds


def tables_of(family, K, L, N, H, seed):
    cfg = ds.make_config(input_dim=16, hidden_dim=H, output_dim=N, hash_family=family, K=K, L=L, bucket_cap=8,
                         max_batch=4, max_labels=4, init_std=0.1, seed=seed, rebuild_period0=0)
    ctx = ds.dslide_init(cfg)
    try:
        off = ds.dslide_get_tensor(ctx, "bucket_off").reshape(L, -1)
        ids = ds.dslide_get_tensor(ctx, "bucket_ids").reshape(L, N)
    finally:
        ds.dslide_destroy(ctx)
    return off, ids


def codes_from_table(off, ids):
    """Invert one table: neuron ids[p] has code b for off[b] <= p < off[b+1]."""
    codes = np.empty(len(ids), dtype=np.uint32)
    codes[ids] = np.repeat(np.arange(len(off) - 1, dtype=np.uint32), np.diff(off))
    return codes


@pytest.mark.parametrize("family,K,N,H", [(1, 6, 50021, 128),                                           # DWTA, 18 bits: two passes
                                           (0, 9, 30011, 64),                                             # 9 bits: one pass
                                           (0, 3, 777, 32)])                                              # tiny, ragged
def test_static_sort_reproduces_the_tables_twice_in_a_row(family, K, N, H):
    L = 2
    off, ids = tables_of(family, K, L, N, H, seed=11)
    bits = int(np.log2(off.shape[1] - 1))
    out_off = torch.full((off.shape[1],), -7, dtype=torch.int32, device="cuda")     # garbage: must be overwritten
    out_ids = torch.full((N,), -7, dtype=torch.int32, device="cuda")
    for t in range(L):                                   # two calls in a row on different data, same scratch
        codes = torch.from_numpy(codes_from_table(off[t], ids[t]).astype(np.int32)).cuda()
        ds.dslide_bucket_sort_static(codes, N, bits, out_off, out_ids)
        torch.cuda.synchronize()
        assert np.array_equal(out_off.cpu().numpy(), off[t])
        assert np.array_equal(out_ids.cpu().numpy(), ids[t])
    # and once more on the first table: the second call's leftovers must not matter either
    codes = torch.from_numpy(codes_from_table(off[0], ids[0]).astype(np.int32)).cuda()
    ds.dslide_bucket_sort_static(codes, N, bits, out_off, out_ids)
    torch.cuda.synchronize()
    assert np.array_equal(out_off.cpu().numpy(), off[0]) and np.array_equal(out_ids.cpu().numpy(), ids[0])


def test_static_sort_rejects_sizes_beyond_its_static_array():
    codes = torch.zeros(8, dtype=torch.int32, device="cuda")
    off = torch.zeros(3, dtype=torch.int32, device="cuda")
    ids = torch.zeros(8, dtype=torch.int32, device="cuda")
    for n, bits in ((ds.STATIC_SORT_MAX_N + 1, 1), (8, ds.STATIC_SORT_MAX_BITS + 1), (8, 0), (-1, 1)):
        with pytest.raises(ds.DslideError) as e:
            ds.dslide_bucket_sort_static(codes, n, bits, off, ids)
        assert e.value.status == ds.ERR_OVERFLOW
    ds.dslide_bucket_sort_static(codes, 8, 1, off, ids)           # still usable; all codes 0 -> one bucket
    torch.cuda.synchronize()
    assert off.cpu().tolist() == [0, 8, 8] and ids.cpu().tolist() == list(range(8))


def reference_sort(codes, bits):
    """An independent statement of the result: stable order of the ids by code, bucket starts by counting."""
    ids = np.argsort(codes, kind="stable").astype(np.int32)
    off = np.zeros((1 << bits) + 1, dtype=np.int32)
    off[1:] = np.cumsum(np.bincount(codes, minlength=1 << bits))
    return off, ids


@pytest.mark.parametrize("n,bits", [(0, 5),                                 # nothing to sort: offsets all zero
                                    (ds.STATIC_SORT_MAX_N if torch.cuda.is_available() else 262144, 18),   # the whole static array, to its last byte
                                    (40001, 10), (40001, 13), (40001, 17),  # second pass narrower than the first
                                    (1, 1), (513, 9)])
def test_static_sort_against_a_stable_argsort(n, bits):
    rng = np.random.default_rng(1000 * bits + n % 997)
    codes = rng.integers(0, 1 << bits, size=n, dtype=np.int64).astype(np.uint32)
    # high garbage bits above `bits` must be ignored
    dirty = (codes | (rng.integers(0, 1 << (31 - bits), size=n, dtype=np.int64).astype(np.uint32) << np.uint32(bits))) if bits < 31 else codes
    want_off, want_ids = reference_sort(codes.astype(np.int64), bits)
    d_codes = torch.from_numpy(dirty.astype(np.int64).astype(np.int32) if n else np.zeros(1, dtype=np.int32)).cuda()
    out_off = torch.full(((1 << bits) + 1,), -7, dtype=torch.int32, device="cuda")
    out_ids = torch.full((max(n, 1),), -7, dtype=torch.int32, device="cuda")
    for rep in range(2):
        ds.dslide_bucket_sort_static(d_codes, n, bits, out_off, out_ids)
        torch.cuda.synchronize()
        assert np.array_equal(out_off.cpu().numpy(), want_off)
        assert np.array_equal(out_ids.cpu().numpy()[:n], want_ids)
