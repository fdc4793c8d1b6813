"""GPU parity: the CUDA path, called through the C ABI, against the CPU checker on the
same seeded inputs.  Integer / byte work (gather, page indexing, tier copies) must be
bit-exact; scores within 1e-4 (fp32 model) or 2e-2 (bf16 model) max-abs."""
import os

import numpy as np
import pytest
import torch

from paper_2601_01712_b200 import synth
from tests.helpers import TOL_BF16, TOL_F32, bf16_noise_bounds, max_abs_err, oracle_model, oracle_scores, small_bf16_shape

pytestmark = pytest.mark.gpu


def _runtime():
    from paper_2601_01712_b200 import binding, runtime
    return binding, runtime


def _setup(shape, seed, batch, hbm_pages=None, host_pages=0, page_ids=None, q_gain=1.0):
    B, rt = _runtime()
    w = synth.make_weights(shape, seed)
    if q_gain != 1.0:                                   # sharper (or flatter) attention logits; a power of two keeps bf16 values exact
        d = shape.d_model
        w.mat["w_qkv"][:, :d, :] *= np.float32(q_gain)
        w.vec["b_qkv"][:, :d] *= np.float32(q_gain)
        if "w_qkv" in w.bits:                           # the bf16 bit patterns are what the device gets
            w.bits["w_qkv"] = synth.round_to_bf16_bits(w.mat["w_qkv"])
    model = rt.Model(shape, w)
    n_pages = [synth.pages_for(batch.prefix_off[i + 1] - batch.prefix_off[i]) for i in range(batch.n_users)]
    total = sum(n_pages)
    pool = rt.KvPool(model, hbm_pages or total + 3, host_pages)
    rows = int(batch.prefix_off[-1] + batch.short_off[-1] + batch.cand_off[-1])
    model.reserve(rows, batch.n_users, total)
    for i in range(batch.n_users):
        pool.alloc(batch.users[i], batch.prefix_off[i + 1] - batch.prefix_off[i], None if page_ids is None else page_ids[i])
    db = rt.DeviceBatch(batch, model.device)
    return w, model, pool, db


def _tiny_batch(shape, seed, p, s, c):
    rng = np.random.default_rng(seed)
    return synth.make_batch(synth.ZipfIds(shape.vocab, 1.1), rng, p, s, c)


# ---------------------------------------------------------------- config 1: tiny fp32 model
def test_config1_fp32_preinfer_rank_full():
    wl = synth.workload(1)
    shape = wl.model
    rng = np.random.default_rng(wl.seed)
    batch = synth.config1_batch(synth.ZipfIds(shape.vocab, wl.zipf_a), rng)
    w, model, pool, db = _setup(shape, wl.seed, batch)
    om = oracle_model(shape, w)

    pool.preinfer(db)
    scores = pool.rank(db)
    full = model.rank_full(db)
    torch.cuda.synchronize()

    # psi: per-layer K / V rows of the prefix
    for i in range(batch.n_users):
        p, _, _ = batch.user_slices(i)
        K, V = om.preinfer(p)
        gK, gV = pool.read_kv(batch.users[i], len(p))
        assert np.max(np.abs(gK.cpu().numpy().astype(np.float64) - K)) <= TOL_F32
        assert np.max(np.abs(gV.cpu().numpy().astype(np.float64) - V)) <= TOL_F32
    want = oracle_scores(om, batch)
    assert max_abs_err(scores.cpu().numpy(), batch, want) <= TOL_F32
    assert max_abs_err(full.cpu().numpy(), batch, want) <= TOL_F32
    # the paper's relation: rank on cache ~= full inference
    assert np.max(np.abs(scores.cpu().numpy() - full.cpu().numpy())) <= TOL_F32
    assert model.launch_count() > 0
    assert model.device_status() == 0
    pool.close(); model.close()


def test_gather_is_bit_exact_fp32_and_bf16():
    _, rt = _runtime()
    for shape in (synth.MODEL_TINY, small_bf16_shape()):
        w = synth.make_weights(shape, 5)
        model = rt.Model(shape, w)
        rng = np.random.default_rng(9)
        ids = synth.ZipfIds(shape.vocab, 1.1).draw(rng, 1000 + 37)
        ids[:3] = [0, shape.vocab - 1, 1]
        out = model.gather(torch.from_numpy(ids).to(model.device))
        torch.cuda.synchronize()
        if shape.dtype == synth.DTYPE_BF16:
            got = out.view(torch.int16).cpu().numpy().view(np.uint16)
            assert np.array_equal(got, w.bits["emb"][ids])
        else:
            assert np.array_equal(out.cpu().numpy().view(np.uint32), w.mat["emb"][ids].view(np.uint32))
        model.close()


# ---------------------------------------------------------------- jagged bf16 batches (several tiles, ragged tails)
JAGGED = [
    ([300, 129, 64, 1000], [5, 0, 70, 33], [130, 7, 0, 257]),
    ([1, 63, 65, 128], [0, 1, 0, 130], [1, 0, 129, 3]),
]


@pytest.mark.parametrize("case", range(len(JAGGED)))
def test_jagged_bf16_matches_checker(case):
    p, s, c = JAGGED[case]
    shape = small_bf16_shape()
    batch = _tiny_batch(shape, 40 + case, p, s, c)
    w, model, pool, db = _setup(shape, 21, batch)
    om = oracle_model(shape, w)
    pool.preinfer(db)
    scores = pool.rank(db)
    full = model.rank_full(db)
    torch.cuda.synchronize()
    for i in range(batch.n_users):
        pp, _, _ = batch.user_slices(i)
        K, V = om.preinfer(pp)
        gK, gV = pool.read_kv(batch.users[i], len(pp))
        assert np.max(np.abs(gK.float().cpu().numpy() - K)) <= 5e-2      # bf16 rows of magnitude ~1-4
        assert np.max(np.abs(gV.float().cpu().numpy() - V)) <= 5e-2
    want = oracle_scores(om, batch)
    assert max_abs_err(scores.cpu().numpy(), batch, want) <= TOL_BF16
    assert max_abs_err(full.cpu().numpy(), batch, want) <= TOL_BF16
    assert model.device_status() == 0
    pool.close(); model.close()


def test_shuffled_page_table_changes_nothing():
    """Pages scattered by a shuffled page table hold bit-identical rows and give bit-identical scores."""
    shape = small_bf16_shape()
    p, s, c = [700, 130, 2049], [17, 64, 3], [140, 200, 31]
    batch = _tiny_batch(shape, 77, p, s, c)
    counts = [synth.pages_for(x) for x in p]
    res = []
    for shuffled in (False, True):
        ids = synth.shuffled_pages(np.random.default_rng(5), sum(counts) + 40, counts) if shuffled else None
        w, model, pool, db = _setup(shape, 22, batch, hbm_pages=sum(counts) + 40, page_ids=ids)
        pool.preinfer(db)
        scores = pool.rank(db)
        torch.cuda.synchronize()
        if shuffled:
            for i in range(batch.n_users):
                assert np.array_equal(pool.pages(batch.users[i]), ids[i])
        kv = [tuple(t.view(torch.int16).cpu().numpy() for t in pool.read_kv(batch.users[i], p[i])) for i in range(3)]
        res.append((scores.cpu().numpy().copy(), kv))
        assert model.device_status() == 0
    pool.close(); model.close()
    assert np.array_equal(res[0][0].view(np.uint32), res[1][0].view(np.uint32))
    for a, b in zip(res[0][1], res[1][1]):
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_preinfer_is_deterministic_and_rank_leaves_pages_untouched():
    shape = small_bf16_shape()
    batch = _tiny_batch(shape, 78, [500, 200], [10, 20], [100, 50])
    w, model, pool, db = _setup(shape, 23, batch)
    pool.preinfer(db)
    torch.cuda.synchronize()
    before = pool.slab.clone()
    pool.rank(db)
    torch.cuda.synchronize()
    assert torch.equal(before, pool.slab)
    # a second pre-infer of the same prefixes into fresh pages gives the same rows
    for u in reversed(batch.users):      # so that the free list hands the same pages out again
        pool.evict(u, False)
    for i, u in enumerate(batch.users):
        pool.alloc(u, batch.prefix_off[i + 1] - batch.prefix_off[i])
    pool.preinfer(db)
    torch.cuda.synchronize()
    assert torch.equal(before, pool.slab)
    assert model.device_status() == 0
    pool.close(); model.close()


def test_batch_equals_single_user_calls_and_candidate_independence():
    B, rt = _runtime()
    shape = small_bf16_shape()
    batch = _tiny_batch(shape, 79, [400, 150], [12, 40], [200, 90])
    w, model, pool, db = _setup(shape, 24, batch)
    pool.preinfer(db)
    scores = pool.rank(db).cpu().numpy().copy()
    # user 1 alone, with only a slice of its candidates
    one = synth.Batch(batch.users[1:2], batch.prefix_ids[400:], np.array([0, 150], np.int32),
                      batch.short_ids[12:], np.array([0, 40], np.int32),
                      batch.cand_ids[200 + 10:200 + 30], np.array([0, 20], np.int32))
    s1 = pool.rank(rt.DeviceBatch(one, model.device)).cpu().numpy()
    assert np.max(np.abs(s1 - scores[200 + 10:200 + 30])) <= 1e-5
    assert model.device_status() == 0
    pool.close(); model.close()


# ---------------------------------------------------------------- boundary behaviour on the device
def test_miss_is_reported_and_nothing_is_enqueued():
    B, rt = _runtime()
    shape = small_bf16_shape()
    batch = _tiny_batch(shape, 80, [100, 100], [4, 4], [8, 8])
    w, model, pool, db = _setup(shape, 25, batch)
    status = np.zeros(2, dtype=np.int32)
    n0 = model.launch_count()
    # users are ALLOCATED but never pre-inferred: rank must refuse
    assert pool.rank(db, per_user_status=status, ok=(B.E_MISS,)) is None
    assert list(status) == [B.TIER_ALLOCATED, B.TIER_ALLOCATED]
    assert model.launch_count() == n0
    pool.preinfer(db)
    unknown = synth.Batch(np.array([0, 99], np.uint64), batch.prefix_ids, batch.prefix_off, batch.short_ids, batch.short_off,
                          batch.cand_ids, batch.cand_off)
    assert pool.rank(rt.DeviceBatch(unknown, model.device), per_user_status=status, ok=(B.E_MISS,)) is None
    assert list(status) == [B.TIER_HBM, B.TIER_MISS]
    # wrong prefix length at pre-infer
    pool.alloc(7, 50)
    bad = synth.Batch(np.array([7], np.uint64), batch.prefix_ids[:60], np.array([0, 60], np.int32), batch.short_ids[:0],
                      np.array([0, 0], np.int32), batch.cand_ids[:0], np.array([0, 0], np.int32))
    assert pool.preinfer(rt.DeviceBatch(bad, model.device), ok=(B.E_INVALID,)) == B.E_INVALID
    assert pool.stats()["misses"] >= 1
    assert model.device_status() == 0
    pool.close(); model.close()


def test_spill_and_reload_round_trip_is_bit_exact():
    B, rt = _runtime()
    shape = small_bf16_shape()
    batch = _tiny_batch(shape, 81, [300, 640], [9, 3], [60, 70])
    w, model, pool, db = _setup(shape, 26, batch, hbm_pages=20, host_pages=20)
    pool.preinfer(db)
    ref_scores = pool.rank(db).cpu().numpy().copy()
    kv0 = [tuple(t.clone() for t in pool.read_kv(u, p)) for u, p in zip(batch.users, (300, 640))]
    side = torch.cuda.Stream()
    for u in batch.users:
        pool.evict(u, True, side)
    assert [pool.lookup(u)[0] for u in batch.users] == [B.TIER_HOST, B.TIER_HOST]
    assert pool.stats()["pages_free"] == 20
    assert pool.rank(db, ok=(B.E_MISS,)) is None
    # scribble over the slab so a reload has to bring the bytes back
    side.synchronize()
    pool.slab.fill_(0x7f)
    for u in batch.users:
        code, ev = pool.reload(u, side)
        assert code == B.OK
        code2, ev2 = pool.reload(u, side)            # single-flight / idempotent
        assert code2 == B.OK
    st = pool.stats()
    assert st["reloads"] == 2 and st["spills"] == 2 and st["reload_bytes"] == st["spill_bytes"]
    scores = pool.rank(db).cpu().numpy()             # rank orders itself behind the reload events
    torch.cuda.synchronize()
    assert np.array_equal(scores.view(np.uint32), ref_scores.view(np.uint32))
    for (k0, v0), u, p in zip(kv0, batch.users, (300, 640)):
        k1, v1 = pool.read_kv(u, p)
        assert torch.equal(k0, k1) and torch.equal(v0, v1)
    assert model.device_status() == 0
    pool.close(); model.close()


# ---------------------------------------------------------------- full-size workloads, sampled users against the checker
def _full_size(workload_index, p_lens, s_lens, c_lens, sample, shuffle):
    """Runs pre-infer + rank + full inference at the sizes and launch configuration the benchmark times, and
    checks the scores of the sampled users (every candidate of theirs) against the checker."""
    from paper_2601_01712_b200 import workloads
    wl = synth.workload(workload_index)
    built = workloads.build(wl.model, wl.seed, p_lens, s_lens, c_lens, n_rotations=1, shuffle_pages=shuffle)
    b, db = built.batches[0], built.dev_batches[0]
    built.pool.preinfer(db)
    scores = built.pool.rank(db).cpu().numpy()
    full = built.model.rank_full(db).cpu().numpy()
    assert built.model.device_status() == 0
    assert np.all(np.isfinite(scores)) and np.all(np.isfinite(full))
    # the attention kernel hands its work items out dynamically (whichever CTA is free takes the next one): the result must
    # not depend on who ran what, so a second run is bit-identical
    again, full_again = built.pool.rank(db).cpu().numpy(), built.model.rank_full(db).cpu().numpy()
    assert np.array_equal(again.view(np.uint32), scores.view(np.uint32))
    assert np.array_equal(full_again.view(np.uint32), full.view(np.uint32))
    # property that holds at any size: rank on cache and full inference agree (the paper's relation)
    assert np.max(np.abs(scores - full)) <= TOL_BF16
    om = oracle_model(wl.model, built.weights)
    want = oracle_scores(om, b, users=sample)
    assert max_abs_err(scores, b, want) <= TOL_BF16
    assert max_abs_err(full, b, want) <= TOL_BF16
    built.pool.close(); built.model.close()


def test_config2_full_size_sampled_users():
    _full_size(2, [2048] * 32, [64] * 32, [512] * 32, sample=[0, 13, 31], shuffle=False)


def test_config3_jagged_full_size_sampled_users():
    wl = synth.workload(3)
    p, s, c = synth.config3_lengths(np.random.default_rng(wl.seed), 128)
    p, s, c = [int(x) for x in p], [int(x) for x in s], [int(x) for x in c]
    order = np.argsort(p)
    sample = [int(order[0]), int(order[40]), int(order[90])]        # a short, a middling and a long prefix
    _full_size(3, p, s, c, sample=sample, shuffle=True)


def test_config4_long_model_sampled_user():
    _full_size(4, [4096] * 16, [128] * 16, [1024] * 16, sample=[5], shuffle=False)


@pytest.mark.parametrize("prefix,user", [(8192, 11), (16384, 3)])
def test_config4_long_prefixes_sampled_user(prefix, user):
    """The long-sequence workload at long prefixes, in the launch configuration the benchmark times (16 users, 8 layers,
    d_model 512): every one of the sampled user's 1024 candidates against the checker.  Longer prefixes are not more of the
    same for the kernels - 130 / 258 key blocks per work item, many more decisions of the stale-maximum softmax, more waves.
    The fp64 checker's pre-infer grows with the square of the prefix: half a minute at 8192 tokens, about two minutes at
    16384 and five at 24576 on 16 host cores, which is why the longest length here is 16384 (the 24576-token case has been
    run with this same function and passes; set RELAYGR_TEST_P24576=1 to include it)."""
    _full_size(4, [prefix] * 16, [128] * 16, [1024] * 16, sample=[user], shuffle=False)


@pytest.mark.skipif(not os.environ.get("RELAYGR_TEST_P24576"), reason="five minutes of CPU checker; opt in with RELAYGR_TEST_P24576=1")
def test_config4_longest_prefix_sampled_user():
    _full_size(4, [24576] * 16, [128] * 16, [1024] * 16, sample=[3], shuffle=False)


def test_reload_tier_workload_small():
    """The reload-tier workload at a reduced population: every call's scores equal those of the same users ranked
    from prefixes that never left HBM (bit for bit: spill and reload move bytes), and the tiers are accounted for."""
    from paper_2601_01712_b200 import tier_workload
    B, rt = _runtime()
    shape = small_bf16_shape()
    report, kept, (model, pool, w, rotations) = tier_workload.run(
        population=48, hbm_users=12, prefix=300, batch=8, n_short=9, n_cand=40, calls=25, warmup=3, shape=shape, collect_scores=True)
    assert report["reloads"] > 0 and report["hit_rate"]["host"] > 0 and report["hit_rate"]["hbm"] > 0
    assert report["spilled_at_start"] == 48 and report["pcie_gb_per_s"] > 0
    pool.close()
    # reference: a pool large enough for everybody, same seeded prefixes (the workload draws them first, in user order)
    rng = np.random.default_rng(synth.BASE_SEED + 5)
    zipf = synth.ZipfIds(shape.vocab, 1.1)
    big = rt.KvPool(model, 48 * synth.pages_for(300))
    for u0 in range(0, 48, 8):
        users = np.arange(u0, u0 + 8, dtype=np.uint64)
        b = synth.make_batch(zipf, rng, [300] * 8, [0] * 8, [0] * 8)
        b.users = users
        for u in users:
            big.alloc(int(u), 300)
        big.preinfer(rt.DeviceBatch(b, model.device))
    so, co = np.arange(9, dtype=np.int32) * 9, np.arange(9, dtype=np.int32) * 40
    for users, rot, got in kept[3:]:
        sid, cid = rotations[rot]
        want = torch.empty(8 * 40, dtype=torch.float32, device=model.device)
        B.relaygr_rank(model.ctx, big.pool, users, sid.data_ptr(), so, cid.data_ptr(), co, want.data_ptr(),
                       torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert torch.equal(got, want)
    assert model.device_status() == 0
    big.close(); model.close()


def test_two_model_slots_share_one_pool():
    """Rank by one context while another context pre-infers other users into the same pool, on two streams: the
    ranked scores are those of an undisturbed run, bit for bit, and match the checker."""
    from paper_2601_01712_b200 import slots_workload
    shape = small_bf16_shape()
    report, scores, batch, w = slots_workload.run(n_rank_users=3, prefix=300, n_short=9, n_cand=40, bg_users=2, bg_prefix=700, calls=12,
                                                  warmup=2, shape=shape, return_scores=True)
    assert report["scores_identical_with_and_without_background"]
    assert report["background_preinfer_calls"] >= 1
    om = oracle_model(shape, w)
    assert max_abs_err(scores, batch, oracle_scores(om, batch)) <= TOL_BF16


# ---------------------------------------------------------------- other widths, edge shapes
@pytest.mark.parametrize("d,heads,ff,layers", [(128, 2, 512, 3), (384, 6, 1536, 2), (1024, 16, 4096, 2)])
def test_other_model_widths_match_checker(d, heads, ff, layers):
    """Widths that take both GEMM shapes (single CTAs where N is not a multiple of 256, CTA pairs elsewhere) and 2 / 6 / 16 heads."""
    shape = small_bf16_shape(vocab=3000, layers=layers, d=d, heads=heads, ff=ff)
    batch = _tiny_batch(shape, 50 + d, [333, 64, 129], [7, 0, 65], [70, 130, 1])
    w, model, pool, db = _setup(shape, 27, batch)
    om = oracle_model(shape, w)
    pool.preinfer(db)
    scores = pool.rank(db).cpu().numpy()
    full = model.rank_full(db).cpu().numpy()
    want = oracle_scores(om, batch)
    assert max_abs_err(scores, batch, want) <= TOL_BF16
    assert max_abs_err(full, batch, want) <= TOL_BF16
    assert model.device_status() == 0
    pool.close(); model.close()


def test_degenerate_batches():
    """No users; users without candidates; one-token prefixes; one user with many candidates over a short prefix (the
    key range is split across CTAs and merged, with the candidates' own keys folded into the first split)."""
    B, rt = _runtime()
    shape = small_bf16_shape()
    # n_users = 0 is accepted and does nothing
    w = synth.make_weights(shape, 28)
    model = rt.Model(shape, w)
    n0 = model.launch_count()
    empty = np.zeros(1, dtype=np.int32)
    B.relaygr_rank_full(model.ctx, 0, None, empty, None, empty, None, empty, None)
    assert model.launch_count() == n0
    model.close()
    # nobody has candidates: nothing to score, but the call is valid
    batch = _tiny_batch(shape, 91, [65, 1], [3, 0], [0, 0])
    w, model, pool, db = _setup(shape, 28, batch)
    pool.preinfer(db)
    out = pool.rank(db)
    assert out.numel() == 0 and model.device_status() == 0
    pool.close(); model.close()
    # prefixes of 1 and 64 tokens, and a long candidate list against a 1500-token prefix (few items -> split key ranges)
    batch = _tiny_batch(shape, 92, [1, 64, 1500], [0, 1, 2], [5, 3, 900])
    w, model, pool, db = _setup(shape, 28, batch)
    om = oracle_model(shape, w)
    pool.preinfer(db)
    scores = pool.rank(db).cpu().numpy()
    full = model.rank_full(db).cpu().numpy()
    want = oracle_scores(om, batch)
    assert max_abs_err(scores, batch, want) <= TOL_BF16
    assert max_abs_err(full, batch, want) <= TOL_BF16
    assert model.device_status() == 0
    pool.close(); model.close()


# ---------------------------------------------------------------- pointwise (HSTU-style) attention
def test_pointwise_attention_fp32_matches_checker():
    """Config-1 batch and model with attn_kind = pointwise: psi, rank on cache and full inference against the checker."""
    import dataclasses
    wl = synth.workload(1)
    shape = dataclasses.replace(wl.model, attn_kind=1)
    rng = np.random.default_rng(wl.seed)
    batch = synth.config1_batch(synth.ZipfIds(shape.vocab, wl.zipf_a), rng)
    w, model, pool, db = _setup(shape, wl.seed, batch)
    om = oracle_model(shape, w)
    pool.preinfer(db)
    scores = pool.rank(db)
    full = model.rank_full(db)
    torch.cuda.synchronize()
    for i in range(batch.n_users):
        p, _, _ = batch.user_slices(i)
        K, V = om.preinfer(p)
        gK, gV = pool.read_kv(batch.users[i], len(p))
        assert np.max(np.abs(gK.cpu().numpy().astype(np.float64) - K)) <= TOL_F32
        assert np.max(np.abs(gV.cpu().numpy().astype(np.float64) - V)) <= TOL_F32
    want = oracle_scores(om, batch)
    assert max_abs_err(scores.cpu().numpy(), batch, want) <= TOL_F32
    assert max_abs_err(full.cpu().numpy(), batch, want) <= TOL_F32
    # and it is a different model from the softmax one
    soft = oracle_scores(oracle_model(wl.model, w), batch, users=[0])
    assert np.max(np.abs(soft[0] - want[0])) > 1e-2
    assert model.device_status() == 0
    pool.close(); model.close()


POINTWISE = [
    ([300, 129, 64, 1000], [5, 0, 70, 33], [130, 7, 0, 257]),      # jagged: ragged tiles, empty segments
    ([1, 63, 65, 128], [0, 1, 0, 130], [1, 0, 129, 3]),
    ([4096], [64], [200]),                                         # one long user: the key range is split and merged
]


@pytest.mark.parametrize("case", range(len(POINTWISE)))
def test_pointwise_attention_bf16_matches_checker(case):
    p, s, c = POINTWISE[case]
    shape = small_bf16_shape(attn_kind=1)
    batch = _tiny_batch(shape, 70 + case, p, s, c)
    w, model, pool, db = _setup(shape, 23, batch)
    om = oracle_model(shape, w)
    pool.preinfer(db)
    scores = pool.rank(db)
    full = model.rank_full(db)
    torch.cuda.synchronize()
    for i in range(batch.n_users):
        pp, _, _ = batch.user_slices(i)
        K, V = om.preinfer(pp)
        gK, gV = pool.read_kv(batch.users[i], len(pp))
        assert np.max(np.abs(gK.float().cpu().numpy() - K)) <= 5e-2
        assert np.max(np.abs(gV.float().cpu().numpy() - V)) <= 5e-2
    want = oracle_scores(om, batch)
    # the variant's scores spread twice as wide as the softmax model's on the same weights and bf16 rounding is relative: the
    # bound follows from the rounding noise this very model and batch must show (helpers.bf16_noise_bounds), not from a run
    max_bound, _, sigma = bf16_noise_bounds(shape, w, batch, want)
    assert max_bound <= 2.5 * TOL_BF16, sigma
    assert max_abs_err(scores.cpu().numpy(), batch, want) <= max_bound
    assert max_abs_err(full.cpu().numpy(), batch, want) <= max_bound
    assert np.std(np.concatenate([v for v in want.values() if len(v)])) > 0.3          # scores are not degenerate
    assert model.device_status() == 0
    pool.close(); model.close()


# ---------------------------------------------------------------- feed-forward widths around the fused kernel's limits
@pytest.mark.parametrize("ff", [128, 2048, 2304])
def test_feed_forward_widths_d256(ff):
    """d_model = 256 with one hidden chunk, with the widest fused feed-forward (2048) and just past it (2304: LayerNorm and
    two GEMM launches instead), on a jagged batch with a ragged last tile."""
    shape = small_bf16_shape(ff=ff)
    batch = _tiny_batch(shape, 90 + ff, [200, 70, 333], [3, 40, 0], [65, 0, 131])
    w, model, pool, db = _setup(shape, 29, batch)
    om = oracle_model(shape, w)
    pool.preinfer(db)
    scores = pool.rank(db)
    full = model.rank_full(db)
    torch.cuda.synchronize()
    want = oracle_scores(om, batch)
    assert max_abs_err(scores.cpu().numpy(), batch, want) <= TOL_BF16
    assert max_abs_err(full.cpu().numpy(), batch, want) <= TOL_BF16
    assert model.device_status() == 0
    pool.close(); model.close()


# ---------------------------------------------------------------- sharp attention logits: the softmax's slow path
@pytest.mark.parametrize("q_gain", [8.0, 64.0])
def test_sharp_logits_take_the_rescaling_path(q_gain):
    """Queries scaled by 8 / 64: logits of tens to hundreds, nearly one-hot softmax rows.  The kernel's exponentials against a
    stale running maximum overflow its row-sum check all the time here, so the block maximum, the rescaling of O and the
    clamps of the FMA-pipe exponential all run.

    What can be asked of the scores: Q and K are stored in bf16 (relative rounding 2^-9), so a logit of magnitude |s| carries an
    absolute error of about |s| * 2^-8, and the softmax weights move by that fraction.  The logits grow with the gain, hence a
    bound of gain * TOL_BF16 against the fp64 checker while the rows are not yet one-hot (gain 8).  At gain 64 a rounding of
    that size decides which of two close keys takes the whole row, so single scores legitimately differ by O(1); there the
    checks are the ones a broken slow path cannot pass: the typical (median) error stays small, and the cached rank and the
    full recompute, which walk the keys in different block and split orders, agree with each other."""
    shape = small_bf16_shape()
    batch = _tiny_batch(shape, 111, [700, 130, 65], [40, 0, 9], [200, 33, 129])
    w, model, pool, db = _setup(shape, 31, batch, q_gain=q_gain)
    om = oracle_model(shape, w)
    pool.preinfer(db)
    scores = pool.rank(db).cpu().numpy()
    full = model.rank_full(db).cpu().numpy()
    torch.cuda.synchronize()
    assert model.device_status() == 0
    want = oracle_scores(om, batch)
    if q_gain <= 8.0:
        assert max_abs_err(scores, batch, want) <= q_gain * TOL_BF16
        assert max_abs_err(full, batch, want) <= q_gain * TOL_BF16
        # the emulation of the unavoidable roundings on these very weights confirms the size of that error (rms about gain x
        # the usual 0.003; its tail is heavier than a normal one here, so it is not used as the bound on the maximum)
        _, rms_bound, sigma = bf16_noise_bounds(shape, w, batch, want)
        err = np.concatenate([scores[batch.cand_off[i]:batch.cand_off[i + 1]] - wv for i, wv in want.items()])
        assert np.sqrt(np.mean(err ** 2)) <= rms_bound, sigma
    else:
        assert np.all(np.isfinite(scores)) and np.all(np.isfinite(full))
        err = np.concatenate([np.abs(scores[batch.cand_off[i]:batch.cand_off[i + 1]] - wv) for i, wv in want.items()])
        assert np.median(err) <= 0.1
    assert np.max(np.abs(scores - full)) <= 4 * TOL_BF16
    pool.close(); model.close()


# ---------------------------------------------------------------- randomized shapes around the tile, page and warp boundaries
_EDGE_LENGTHS = [1, 2, 31, 32, 33, 63, 64, 65, 127, 128, 129, 191, 192, 193, 255, 256, 257, 511, 512, 513, 1023, 1024, 1025]


def _random_case(rng):
    def pick(lo, hi, allow_zero=False):
        r = rng.random()
        if allow_zero and r < 0.15:
            return 0
        if r < 0.5:
            return int(rng.choice([e for e in _EDGE_LENGTHS if lo <= e <= hi]))
        return int(rng.integers(lo, hi + 1))
    d = int(rng.choice([128, 256, 256, 256, 384, 512]))
    layers = int(rng.integers(1, 4))
    ff = int(rng.choice([128, 256, 512, 1024])) if d == 256 else (4 * d if rng.random() < 0.5 else int(rng.choice([128, 384, 640])))
    kind = int(rng.random() < 0.25)
    n = int(rng.integers(1, 6))
    return d, layers, ff, kind, [pick(1, 1300) for _ in range(n)], [pick(1, 200, True) for _ in range(n)], [pick(1, 300, True) for _ in range(n)]


@pytest.mark.parametrize("block", range(4))
def test_randomized_shapes_match_checker(block):
    """Seeded random models (width, depth, feed-forward width, attention variant) and jagged batches whose lengths cluster
    around the boundaries of the 64-token pages, the 128-row query tiles and the 32-row warps, half of them on shuffled
    pages.  The named workloads' bound (2e-2) is not a bound for every shape: the rounding a bf16 model cannot avoid gives
    single-layer and narrow models score errors of rms up to 0.0065, whose largest of several hundred reaches 0.02 in a pure
    numpy emulation with no kernel in it.  Each case is therefore held to the bounds derived from that emulation for its own
    model and batch (helpers.bf16_noise_bounds): maximum <= max(2e-2, 5 sigma), rms <= 1.5 sigma."""
    rng = np.random.default_rng(9100 + block)
    for it in range(6):
        d, layers, ff, kind, p, s, c = _random_case(rng)
        shape = small_bf16_shape(vocab=3000, layers=layers, d=d, heads=d // 64, ff=ff, attn_kind=kind)
        batch = _tiny_batch(shape, 1000 * block + it, p, s, c)
        counts = [synth.pages_for(x) for x in p]
        ids = synth.shuffled_pages(np.random.default_rng(it), sum(counts) + 7, counts) if rng.random() < 0.5 else None
        w, model, pool, db = _setup(shape, 500 + 10 * block + it, batch, hbm_pages=sum(counts) + 7, page_ids=ids)
        om = oracle_model(shape, w)
        pool.preinfer(db)
        scores = pool.rank(db).cpu().numpy()
        full = model.rank_full(db).cpu().numpy()
        torch.cuda.synchronize()
        assert model.device_status() == 0
        want = oracle_scores(om, batch)
        max_bound, rms_bound, sigma = bf16_noise_bounds(shape, w, batch, want)
        case = (d, layers, ff, kind, p, s, c, sigma)
        assert max_bound <= 2.5 * TOL_BF16, case                 # the yardstick itself stays in a sane range
        for got in (scores, full):
            assert max_abs_err(got, batch, want) <= max_bound, case
            err = np.concatenate([got[batch.cand_off[i]:batch.cand_off[i + 1]] - wv for i, wv in want.items()])
            if len(err):
                assert np.sqrt(np.mean(err ** 2)) <= rms_bound, case
        pool.close(); model.close()
