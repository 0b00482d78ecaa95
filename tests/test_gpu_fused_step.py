"""GPU: the one-launch accept-and-fill against the two calls it replaces and against the oracle.

The fused call has to give what xg_accept_token followed by xg_fill_next_token_bitmask gives:
the same statuses, the same matcher state and the same mask words, for accepted tokens, rejected
tokens, end of sequence (with and without restart) and terminated requests.
"""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2601_04426_b200 import inputs
from test_gpu_parity import _engine, _oracle_side, _run_trajectories

pytestmark = pytest.mark.gpu

XG_ERR_TOKEN_REJECTED, XG_ERR_TERMINATED = -7, -8


@pytest.mark.parametrize("name,kw,check", [
    ("C1", {}, None),
    ("C3", {"batch": 16, "steps": 48}, {0, 5, 17, 33, 47}),
    ("C4", {"batch": 6, "steps": 120}, {0, 1, 30, 60, 119}),
    ("C5", {"batch": 8, "steps": 64}, {0, 7, 31, 63}),
    ("R256", {"batch": 4, "steps": 120, "vocab_size": 16384}, {0, 40, 80, 119}),
])
def test_fused_steps_bit_exact_against_the_oracle(name, kw, check):
    w = inputs.make_workload(name, **kw)
    steps = check if check is not None else set(range(w.steps))
    assert _run_trajectories(w, steps, check_requests={1} if w.batch > 1 else None, fused=True) >= len(steps)


@pytest.mark.parametrize("name,kw,check", [
    ("C1", {}, None),
    ("C5", {"batch": 8, "steps": 64}, {0, 7, 31, 63}),
])
def test_accept_with_restart_at_end_of_sequence_bit_exact(name, kw, check):
    """The separate accept call with its restart option: no reset call, same masks."""
    w = inputs.make_workload(name, **kw)
    steps = check if check is not None else set(range(w.steps))
    assert _run_trajectories(w, steps, check_requests={1} if w.batch > 1 else None, restart=True) >= len(steps)


def test_fused_equals_accept_then_fill_word_for_word():
    """Two sessions over the same workload, one stepping with the fused call and one with the two
    separate calls (and a reset at end of sequence): every mask row and status agrees at every step."""
    torch, engine = _engine()
    w = inputs.make_workload("C5", batch=12, steps=96)
    a, b = engine.Session(w), engine.Session(w)
    try:
        a.fill(); b.fill()
        for step in range(w.steps):
            assert np.array_equal(a.mask_numpy(), b.mask_numpy()), step
            toks = [w.trajectories[r][step] for r in range(a.n)]
            a.accept_fill(toks, restart_on_eos=True)
            b.accept(toks)
            for r in range(b.n):
                if toks[r] == w.vocab.eos_id:
                    b.reset(r)
            b.fill()
            assert (a.accept_status.cpu().numpy() == 0).all() and (b.accept_status.cpu().numpy() == 0).all()
            assert np.array_equal(a.status.cpu().numpy(), b.status.cpu().numpy())
        assert np.array_equal(a.mask_numpy(), b.mask_numpy())
    finally:
        a.close(); b.close()


def test_rejected_token_keeps_state_and_mask():
    torch, engine = _engine()
    w = inputs.make_workload("C3", batch=8, steps=24)
    s = engine.Session(w)
    ov, _, oms = _oracle_side(w)
    try:
        s.fill()
        for step in range(10):
            toks = [w.trajectories[r][step] for r in range(s.n)]
            s.accept_fill(toks)
            for r in range(s.n):
                assert oms[r].accept_token(ov, toks[r]) == 1
        before = s.mask_numpy().copy()
        # one disallowed token for the even requests, the trajectory's token for the odd ones
        toks = []
        for r in range(s.n):
            if r % 2 == 0:
                row = O.unpack_bits(before[r], ov.size)
                toks.append(int(np.nonzero(~row)[0][0]))
            else:
                toks.append(w.trajectories[r][10])
        s.accept_fill(toks)
        ast = s.accept_status.cpu().numpy()
        after = s.mask_numpy()
        for r in range(s.n):
            if r % 2 == 0:
                assert ast[r] == XG_ERR_TOKEN_REJECTED
                assert np.array_equal(after[r], before[r])
            else:
                assert ast[r] == 0 and oms[r].accept_token(ov, toks[r]) == 1
                assert np.array_equal(after[r], oms[r].mask(ov))
        assert (s.status.cpu().numpy() == 0).all()
        # the rejected requests carry on from where they were
        toks = [w.trajectories[r][10 if r % 2 == 0 else 11] for r in range(s.n)]
        s.accept_fill(toks)
        assert (s.accept_status.cpu().numpy() == 0).all()
        for r in range(s.n):
            assert oms[r].accept_token(ov, toks[r]) == 1
            assert np.array_equal(s.mask_numpy()[r], oms[r].mask(ov))
    finally:
        s.close()


def test_end_of_sequence_without_restart_terminates():
    torch, engine = _engine()
    w = inputs.make_workload("C5", batch=12, steps=96)
    s = engine.Session(w)
    ov, _, oms = _oracle_side(w)
    try:
        s.fill()
        done = [False] * s.n
        saw_eos = 0
        for step in range(w.steps):
            toks = [w.trajectories[r][step] for r in range(s.n)]
            s.accept_fill(toks)                      # no restart: the request terminates at EOS
            ast, fst, mask = s.accept_status.cpu().numpy(), s.status.cpu().numpy(), s.mask_numpy()
            for r in range(s.n):
                if done[r]:
                    assert ast[r] == XG_ERR_TERMINATED and fst[r] == XG_ERR_TERMINATED and not mask[r].any()
                    continue
                assert ast[r] == 0
                if oms[r].accept_token(ov, toks[r]) == 2:
                    done[r] = True
                    saw_eos += 1
                    assert s.matchers[r].is_terminated()
                    assert fst[r] == XG_ERR_TERMINATED and not mask[r].any()
                else:
                    assert fst[r] == 0
                    if step % 8 == 0:
                        assert np.array_equal(mask[r], oms[r].mask(ov))
        assert saw_eos >= 1
        # a reset brings a terminated request back
        r = done.index(True)
        s.reset(r); oms[r].reset()
        s.fill()
        assert np.array_equal(s.mask_numpy()[r], oms[r].mask(ov))
    finally:
        s.close()
