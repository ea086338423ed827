"""GPU-vs-oracle parity of the LSH-sampled hidden layer (Algorithm 1: active neurons are retrieved for every layer;
Section 3.6: the second kind of layer).  Projections, tables over the hidden neurons, codes of the inputs and active
masks bit-exact; activations exactly 0 for neurons that were not retrieved and bit-exact otherwise; the rest of the
step at the usual bars; weights of the first layer that no sample touched (input zero, or neuron not retrieved) bit-
identical after the update."""
import numpy as np
import pytest
import torch

from tests.helpers import max_rel_err

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2201_12667_b200 import binding as ds
    from paper_2201_12667_b200 import workloads
    from tests.gpu_harness import Pair
    from tests.test_gpu_parity import ACT_TOL, W_TOL, compare_forward, compare_weights

SIMHASH, DWTA = 0, 1


def mask_bits(words, H):
    """[B][Hw] u32 -> [B][H] 0/1"""
    B = words.shape[0]
    return ((words[:, :, None] >> np.arange(32, dtype=np.uint32)[None, None, :]) & 1).reshape(B, -1)[:, :H].astype(np.uint8)


@pytest.mark.parametrize("H,hK,hL,hcap,family", [(128, 3, 6, 12, DWTA), (64, 2, 5, 8, SIMHASH), (256, 4, 16, 16, DWTA), (1024, 5, 12, 24, DWTA)])
def test_sampled_hidden_layer_step(H, hK, hL, hcap, family):
    c = workloads.config("mid")
    pr = Pair(D=c["D"], H=H, N=8009, family=family, K=3, L=6, bucket_cap=16, max_batch=24, max_labels=16, lr=1e-3, seed=3,
              hidden_K=hK, hidden_L=hL, hidden_cap=hcap, sync_weights=False)
    try:
        # the library's own draw of the projections and its tables over its own initial weights
        assert np.array_equal(ds.dslide_get_tensor(pr.ctx, "proj1"), pr.o.get("proj1"))
        pr.push_state()
        assert np.array_equal(ds.dslide_get_tensor(pr.ctx, "bucket1_off"), pr.o.get("bucket1_off"))
        assert np.array_equal(ds.dslide_get_tensor(pr.ctx, "bucket1_ids"), pr.o.get("bucket1_ids"))
        wl = workloads.Workload(workloads.config("mid", N=8009), seed=12)
        before = {n: ds.dslide_get_tensor(pr.ctx, n) for n in ("W1", "mW1", "vW1", "b1")}
        for i in range(2):
            batch = wl.batch(i, batch_size=24)
            B = 24
            lo = pr.o.train_step(*batch)
            lg = pr.gpu_step(batch)
            tol = ACT_TOL if i == 0 else W_TOL
            assert abs(lo - lg) <= tol * abs(lo), (i, lo, lg)
            hact = pr.o.get("hact").reshape(B, H)
            if i == 0:
                assert np.array_equal(ds.dslide_get_last(pr.ctx, "codes1", B), pr.o.get("codes1").reshape(B, hL))
                assert np.array_equal(mask_bits(ds.dslide_get_last(pr.ctx, "hidden_mask", B), H), hact)
                assert 0.02 < hact.mean() < 0.98
                h = ds.dslide_get_last(pr.ctx, "hidden", B)
                assert np.all(h[hact == 0] == 0)
            compare_forward(pr, batch, bit_exact_hidden=(i == 0), tol=tol)
            if i == 0:
                touched = np.zeros((pr.D, H), dtype=bool)
                for s in range(B):
                    touched[batch[1][batch[0][s]:batch[0][s + 1]]] |= hact[s].astype(bool)
                for n in ("W1", "mW1", "vW1"):
                    a, b = before[n].reshape(pr.D, H), ds.dslide_get_tensor(pr.ctx, n).reshape(pr.D, H)
                    assert np.array_equal(a[~touched].view(np.uint32), b[~touched].view(np.uint32)), n
                    assert not np.array_equal(a[touched], b[touched])
                off = ~hact.any(axis=0).astype(bool)
                assert np.array_equal(before["b1"][off].view(np.uint32), ds.dslide_get_tensor(pr.ctx, "b1")[off].view(np.uint32))
        compare_weights(pr)
        # a rebuild redraws the projections and rebuilds the hidden layer's tables too
        ds.dslide_rebuild_tables(pr.ctx)
        ds.dslide_sync(pr.ctx)
        pr.o.rebuild_tables()
        assert np.array_equal(ds.dslide_get_tensor(pr.ctx, "proj1"), pr.o.get("proj1"))
        # the tables depend on the signs of sums over each side's own weights (equal within the weight bar only)
        go, oo = ds.dslide_get_tensor(pr.ctx, "bucket1_off"), pr.o.get("bucket1_off")
        assert go.shape == oo.shape and go.reshape(hL, -1)[:, -1].tolist() == [H] * hL
    finally:
        pr.close()


def test_sampled_hidden_layer_predict():
    c = workloads.config("mid")
    pr = Pair(D=c["D"], H=128, N=8009, family=DWTA, K=3, L=6, bucket_cap=16, max_batch=24, max_labels=16, lr=1e-3, seed=4,
              hidden_K=3, hidden_L=6, hidden_cap=12)
    try:
        wl = workloads.Workload(workloads.config("mid", N=8009), seed=13)
        batch = wl.batch(0, batch_size=24)
        dev = [torch.from_numpy(a).cuda() for a in batch[:3]]
        for dense in (0, 1):
            out_ids = torch.zeros(24 * 5, dtype=torch.int32, device="cuda")
            out_sc = torch.zeros(24 * 5, dtype=torch.float32, device="cuda")
            ds.dslide_predict_topk(pr.ctx, 24, dev[0], dev[1], dev[2], 5, dense, out_ids, out_sc)
            ds.dslide_sync(pr.ctx)
            ids_o, sc_o = pr.o.predict_topk(batch[0], batch[1], batch[2], 5, dense=bool(dense))
            assert np.array_equal(out_ids.cpu().numpy().reshape(24, 5), ids_o)
            assert max_rel_err(out_sc.cpu().numpy().reshape(24, 5), sc_o, 1e-2) < ACT_TOL
    finally:
        pr.close()
