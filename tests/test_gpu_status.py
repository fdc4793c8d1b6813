"""The device status word (relaygr_device_status): reported, stops the tensor-core kernels of later calls, cleared by
relaygr_set_workspace, set by a token id outside the table, forwarded by relaygr_rank_full_static.  The word is written
from the host or set by a kernel's own bounds check: no kernel is made to misbehave."""
import numpy as np
import pytest
import torch

from paper_2601_01712_b200 import synth
from tests.helpers import small_bf16_shape

pytestmark = pytest.mark.gpu


def _built(seed=5):
    from paper_2601_01712_b200 import workloads
    return workloads.build(small_bf16_shape(), seed, [200, 130], [9, 32], [40, 150], n_rotations=1)


def test_status_word_is_reported_stops_tensor_kernels_and_is_cleared():
    from paper_2601_01712_b200 import binding as B
    from paper_2601_01712_b200 import workloads
    built = _built()
    model, pool, db = built.model, built.pool, built.dev_batches[0]
    pool.preinfer(db)
    want = pool.rank(db).clone()
    torch.cuda.synchronize()
    assert model.device_status() == 0
    pages_ok = pool.slab.clone()

    # a non-zero word, written from the host
    model._ws[:4].copy_(torch.tensor([7, 0, 0, 0], dtype=torch.uint8))
    workloads.realloc_users(built)
    pool.slab.fill_(0x5A)
    pool.preinfer(db)                                       # the projections' epilogues write K/V pages: they must not run
    torch.cuda.synchronize()
    assert bool(torch.all(pool.slab == 0x5A)), "a tensor-core kernel ran although the status word was set"
    assert model.device_status() == 7                       # the first code stays, and is reported
    pool.rank(db)
    assert model.device_status() == 7

    # lending the workspace again clears the word; the path then works as before, bit for bit
    B.relaygr_set_workspace(model.ctx, model._ws.data_ptr(), model._ws.numel())
    assert model.device_status() == 0
    workloads.realloc_users(built)
    pool.preinfer(db)
    got = pool.rank(db)
    torch.cuda.synchronize()
    assert model.device_status() == 0
    assert torch.equal(got, want)
    assert torch.equal(pool.slab, pages_ok)
    pool.close(); model.close()


def test_token_id_outside_the_table_is_recorded_not_clamped_silently():
    from paper_2601_01712_b200 import binding as B
    built = _built(6)
    model, pool, db = built.model, built.pool, built.dev_batches[0]
    vocab = built.shape.vocab
    pool.preinfer(db)
    pool.rank(db)
    assert model.device_status() == 0
    # the gather entry point: one bad id among good ones; every access stays inside the table
    ids = torch.tensor([3, vocab + 5, 7, -2], dtype=torch.int32, device=model.device)
    out = model.gather(ids)
    assert model.device_status() == B.DEVSTATUS_BAD_INDEX
    table = model._t["emb"]
    assert torch.equal(out[0], table[3]) and torch.equal(out[2], table[7])
    assert torch.equal(out[1], table[vocab - 1]) and torch.equal(out[3], table[0])
    B.relaygr_set_workspace(model.ctx, model._ws.data_ptr(), model._ws.numel())
    assert model.device_status() == 0
    # the hot path: a candidate id past the table
    bad = db.cand_ids.clone()
    db.cand_ids[5] = vocab
    pool.rank(db)
    assert model.device_status() == B.DEVSTATUS_BAD_INDEX
    db.cand_ids.copy_(bad)
    B.relaygr_set_workspace(model.ctx, model._ws.data_ptr(), model._ws.numel())
    pool.rank(db)
    assert model.device_status() == 0
    pool.close(); model.close()


def test_static_entry_point_forwards_its_status_word():
    from paper_2601_01712_b200 import binding as B
    built = _built(7)
    model, db = built.model, built.dev_batches[0]
    stream = torch.cuda.current_stream().cuda_stream
    scores = torch.zeros(int(db.cand_off[-1]), dtype=torch.float32, device=model.device)

    def call():
        B.relaygr_rank_full_static(model.ctx, db.n_users, db.prefix_ids.data_ptr(), db.prefix_off, db.short_ids.data_ptr(),
                                   db.short_off, db.cand_ids.data_ptr(), db.cand_off, scores.data_ptr(), stream)

    call()
    assert model.device_status() == 0
    good = scores.clone()
    keep = db.prefix_ids.clone()
    db.prefix_ids[11] = built.shape.vocab + 1              # the built-in array's own status word records it ...
    call()
    assert model.device_status() == B.DEVSTATUS_BAD_INDEX   # ... and it reaches the word relaygr_device_status reads
    db.prefix_ids.copy_(keep)
    B.relaygr_set_workspace(model.ctx, model._ws.data_ptr(), model._ws.numel())
    call()                                                  # the array's word starts clean on every call
    assert model.device_status() == 0
    assert torch.equal(scores, good)
    built.pool.close(); model.close()
