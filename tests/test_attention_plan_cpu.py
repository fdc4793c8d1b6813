"""The attention work list (host logic of the library, no GPU): whatever the split policy decides, every key block of
every (user, head, 128-row tile) is covered exactly once, split pieces own distinct partial slots and are merged once,
and the candidates' own keys are folded in by exactly one piece (paper Section 3.2: candidates see the prefix, the
short-term tokens and themselves)."""
import numpy as np
import pytest

from paper_2601_01712_b200 import binding as B

SMS = 148


def tiles_of(mode, P, S, C):
    """(q0, n_q, number of visible 64-key blocks) of each 128-row tile of one user, from the mask's definition."""
    if mode == 0:
        n_q, q_pos0, n_paged, n_lin, lin_pos0, causal_end = P, 0, P, 0, P, P
    elif mode == 1:
        n_q, q_pos0, n_paged, n_lin, lin_pos0, causal_end = S + C, P, P, S, P, P + S
    else:
        n_q, q_pos0, n_paged, n_lin, lin_pos0, causal_end = P + S + C, 0, 0, P + S, 0, P + S
    out = []
    for q0 in range(0, n_q, 128):
        nq = min(128, n_q - q0)
        last = q_pos0 + q0 + nq - 1
        kmax = last if last < causal_end else causal_end - 1        # last key position any row of the tile sees
        nb = 0
        if kmax >= 0:
            # blocks: the pages of the cached prefix first, then 64-row groups of the call's own (linear) keys
            vis_paged = min(n_paged, kmax + 1)
            nb = (vis_paged + 63) // 64
            if vis_paged == n_paged and n_lin > 0 and kmax >= lin_pos0:
                nb += (min(n_lin, kmax - lin_pos0 + 1) + 63) // 64
        out.append((q0, nq, nb, q_pos0 + q0 + nq > causal_end))
    return out


def check_plan(mode, Ps, Ss, Cs, H, sms=SMS):
    items, merges = B.relaygr_attention_plan(mode, Ps, Ss, Cs, H, sms)
    want = {}
    for u, (P, S, C) in enumerate(zip(Ps, Ss, Cs)):
        for q0, nq, nb, has_cand in tiles_of(mode, P, S, C):
            for h in range(H):
                want[(u, h, q0)] = (nq, nb, has_cand)
    cover = {k: np.zeros(v[1], dtype=np.int32) for k, v in want.items()}
    selfs = {k: 0 for k in want}
    pieces = {k: [] for k in want}
    slots = set()
    for u, h, q0, nq, b0, b1, slot, with_self in items.tolist():
        key = (u, h, q0)
        assert key in want and want[key][0] == nq
        assert 0 <= b0 <= b1 <= want[key][1]
        cover[key][b0:b1] += 1
        selfs[key] += with_self
        pieces[key].append(slot)
        if slot >= 0:
            assert slot not in slots
            slots.add(slot)
    for key, (nq, nb, has_cand) in want.items():
        assert (cover[key] == 1).all(), key
        assert selfs[key] == (1 if has_cand else 0), key
        assert len(pieces[key]) >= 1
        if len(pieces[key]) > 1:
            assert all(s >= 0 for s in pieces[key])
        else:
            assert pieces[key] == [-1]
    merged = {}
    for u, h, q0, nq, slot0, ns in merges.tolist():
        key = (u, h, q0)
        assert key not in merged and ns >= 2
        merged[key] = sorted(range(slot0, slot0 + ns))
    for key, sl in pieces.items():
        if len(sl) > 1:
            assert merged.get(key) == sorted(sl), key
        else:
            assert key not in merged
    return items, merges


@pytest.mark.parametrize("mode", [0, 1, 2])
def test_plan_covers_every_block_once(mode):
    rng = np.random.default_rng(5 + mode)
    for trial in range(12):
        n = int(rng.integers(1, 40))
        Ps = rng.integers(0, 5000, size=n).tolist()
        Ss = rng.integers(0, 200, size=n).tolist()
        Cs = rng.integers(0, 700, size=n).tolist()
        if trial == 0:
            Ps[0], Ss[0], Cs[0] = 0, 0, 1
        check_plan(mode, Ps, Ss, Cs, int(rng.choice([1, 4, 8])))


def test_plan_empty_and_degenerate():
    items, merges = B.relaygr_attention_plan(1, [], [], [], 4, SMS)
    assert len(items) == 0 and len(merges) == 0
    check_plan(1, [0], [0], [1], 4)              # a candidate with nothing before it: no key blocks, its own key only
    check_plan(0, [1], [0], [0], 4)
    check_plan(1, [64], [0], [0], 4)             # no query rows at all


def test_tail_of_the_list_is_split_to_fill_the_last_wave():
    """32 users x 2048-token prefix, 64 short-term and 512 candidate tokens, 4 heads: 640 equal items on 296 slots.  Two
    full waves stay whole; the 48 items left over are split so that their pieces occupy (most of) one more wave."""
    items, merges = check_plan(1, [2048] * 32, [64] * 32, [512] * 32, 4)
    whole = items[items[:, 6] < 0]
    split = items[items[:, 6] >= 0]
    assert len(whole) == 592 and (whole[:, 5] - whole[:, 4] == 33).all()
    assert len(merges) == 48
    assert 148 < len(split) <= 296
    assert (items[:592, 6] < 0).all()            # the split pieces come last in launch order
    n_blocks = split[:, 5] - split[:, 4]
    assert n_blocks.min() >= 4 and n_blocks.max() - n_blocks.min() <= 1


def test_few_items_are_split_to_fill_the_gpu_and_many_are_not():
    items, merges = check_plan(1, [2048], [64], [512], 4)           # one request: 20 tiles x heads on 296 slots
    assert len(merges) == 20 and 100 <= len(items) <= 296
    items, merges = check_plan(0, [2048] * 32, [0] * 32, [0] * 32, 4)       # 2048 causal tiles: several waves, nothing left to gain
    assert len(items) >= 2048 and len(merges) <= 64
    # a launch that already fills whole waves is left alone
    items, merges = check_plan(1, [2048] * 37, [0] * 37, [256] * 37, 4)     # 37 x 2 x 4 = 296 items
    assert len(items) == 296 and len(merges) == 0
