"""relaygr_rank_full_static: full inference whose scratch is an array built into the library.

Some users of the library cannot allocate device memory when a request arrives - all of
the GPU's memory was handed out at start-up, or they run inside another framework's pool, or
they sit on a latency-critical thread where an allocation's device synchronisation is not
acceptable - and have no workspace to lend either.  This entry point gives them the miss
fallback all the same.  The test calls it through the C ABI, twice in a row with different
batches (the array keeps the previous call's contents), and compares with relaygr_rank_full
on a lent workspace.  It lives in a file of its own that pytest collects last.
"""
import numpy as np
import pytest
import torch

from paper_2601_01712_b200 import synth
from tests.helpers import TOL_BF16, TOL_F32, small_bf16_shape

pytestmark = pytest.mark.gpu


def _scores_static(B, model, db):
    out = torch.full((int(db.cand_off[-1]),), float("nan"), dtype=torch.float32, device=model.device)
    B.relaygr_rank_full_static(model.ctx, db.n_users, db.prefix_ids.data_ptr(), db.prefix_off, db.short_ids.data_ptr(),
                               db.short_off, db.cand_ids.data_ptr(), db.cand_off, out.data_ptr(),
                               torch.cuda.current_stream().cuda_stream)
    return out


@pytest.mark.parametrize("kind", ["bf16", "fp32"])
def test_static_scratch_matches_lent_workspace_on_two_calls_in_a_row(kind):
    from paper_2601_01712_b200 import binding as B
    from paper_2601_01712_b200 import runtime as rt
    shape, tol = (small_bf16_shape(), TOL_BF16) if kind == "bf16" else (synth.MODEL_TINY, TOL_F32)
    w = synth.make_weights(shape, 31)
    zipf = synth.ZipfIds(shape.vocab, 1.1)
    rng = np.random.default_rng(90)
    # the second batch is smaller and shaped differently, so it runs over the first call's leftovers
    batches = [synth.make_batch(zipf, rng, [700, 130, 65], [20, 0, 64], [150, 40, 7]),
               synth.make_batch(zipf, rng, [90, 300], [3, 33], [64, 129])]

    # reference: the existing entry point on a workspace lent by the caller
    ref_model = rt.Model(shape, w)
    ref_model.reserve(max(int(b.prefix_off[-1] + b.short_off[-1] + b.cand_off[-1]) for b in batches), 3, 0)
    want = [ref_model.rank_full(rt.DeviceBatch(b, ref_model.device)).cpu().numpy().copy() for b in batches]
    assert ref_model.device_status() == 0
    ref_model.close()

    # the static entry point on a context that was never lent a workspace
    model = rt.Model(shape, w)
    for b, expect in zip(batches, want):
        got = _scores_static(B, model, rt.DeviceBatch(b, model.device))
        torch.cuda.synchronize()
        got = got.cpu().numpy()
        assert np.all(np.isfinite(got))
        assert float(np.max(np.abs(got - expect))) <= tol
    # a lent workspace is left alone (beyond its status word), and receives the (healthy) status
    model.reserve(64, 1, 0)
    model._ws[1024:].fill_(0xA7)
    db1, db0 = rt.DeviceBatch(batches[1], model.device), rt.DeviceBatch(batches[0], model.device)
    got = _scores_static(B, model, db1)
    assert model.device_status() == 0
    assert float(np.max(np.abs(got.cpu().numpy() - want[1]))) <= tol
    assert bool(torch.all(model._ws[1024:] == 0xA7)), "the lent workspace was written"
    # nothing is allocated on the device by a call (the set-up of the first call is over by now), and two calls queued
    # back to back on one stream without a synchronisation in between share the array in order
    torch.cuda.synchronize()
    free0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    out0 = torch.full((int(db0.cand_off[-1]),), float("nan"), dtype=torch.float32, device=model.device)
    out1 = torch.full((int(db1.cand_off[-1]),), float("nan"), dtype=torch.float32, device=model.device)
    free1, alloc1 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    s = torch.cuda.current_stream().cuda_stream
    for db, out in ((db0, out0), (db1, out1)):
        B.relaygr_rank_full_static(model.ctx, db.n_users, db.prefix_ids.data_ptr(), db.prefix_off, db.short_ids.data_ptr(),
                                   db.short_off, db.cand_ids.data_ptr(), db.cand_off, out.data_ptr(), s)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free1 and torch.cuda.memory_allocated() == alloc1
    assert free1 <= free0 and alloc1 >= alloc0
    assert float(np.max(np.abs(out0.cpu().numpy() - want[0]))) <= tol
    assert float(np.max(np.abs(out1.cpu().numpy() - want[1]))) <= tol
    model.close()


def test_static_scratch_rejects_batches_beyond_its_size():
    from paper_2601_01712_b200 import binding as B
    from paper_2601_01712_b200 import runtime as rt
    shape = small_bf16_shape()
    model = rt.Model(shape, synth.make_weights(shape, 32))
    rows = 40_000                                    # far more activations than the built-in array holds
    assert B.relaygr_workspace_bytes(model.ctx, rows, 1, 0) > B.STATIC_SCRATCH_BYTES
    ids = torch.zeros(rows, dtype=torch.int32, device=model.device)
    off = np.array([0, rows], np.int32)
    zero = np.array([0, 0], np.int32)
    n0 = model.launch_count()
    with pytest.raises(B.RelayGRError) as e:
        B.relaygr_rank_full_static(model.ctx, 1, ids.data_ptr(), off, ids.data_ptr(), zero, ids.data_ptr(), zero, 0,
                                   torch.cuda.current_stream().cuda_stream)
    assert e.value.code == B.E_NOSPACE and "built-in array" in str(e.value)
    assert model.launch_count() == n0                # nothing was enqueued
    model.close()
