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


@pytest.mark.parametrize("name,kw", [
    ("C1", {}),                                            # fp32, one request
    ("C3", {"batch": 16, "steps": 48}),                    # bf16, a grammar per request
    ("C4", {"batch": 6, "steps": 60}),                     # fp32, free text (almost nothing masked) and tool calls
    ("C5", {"batch": 8, "steps": 40}),                     # bf16, many uncertain tokens
])
def test_fill_and_apply_in_one_launch_equals_the_two_calls(name, kw):
    """xg_fill_and_apply_token_bitmask against xg_fill_next_token_bitmask + xg_apply_token_bitmask and against
    the oracle: mask words, statuses and every logit of the batch, with a padded logits stride; a terminated
    request's row becomes all -inf."""
    torch, engine = _engine()
    w = inputs.make_workload(name, **kw)
    s = engine.Session(w)
    ov, _, oms = _oracle_side(w)
    n, V = s.n, w.vocab.size
    elt_per_16 = 4 if w.dtype == "f32" else 8
    stride = (V + elt_per_16 - 1) // elt_per_16 * elt_per_16 + elt_per_16      # one vector of padding behind every row
    raw = (lambda a: a.view(np.uint32)) if w.dtype == "f32" else (lambda a: a)
    pad_value = np.float32(7.0) if w.dtype == "f32" else np.uint16(0x40E0)
    try:
        for step in range(w.steps):
            logits_np = np.full((n, stride), pad_value, dtype=np.float32 if w.dtype == "f32" else np.uint16)
            logits_np[:, :V] = inputs.make_logits(w.logits_seed + step, n, V, w.dtype)
            fused = engine.logits_tensor(logits_np, s.device)
            s.fill_apply(fused[:, :])
            mask_fused, status_fused = s.mask_numpy().copy(), s.status.cpu().numpy().copy()
            two = engine.logits_tensor(logits_np, s.device)
            s.fill()
            s.apply(two)
            assert np.array_equal(mask_fused, s.mask_numpy()) and np.array_equal(status_fused, s.status.cpu().numpy()), step
            got = engine.logits_numpy(fused)
            assert np.array_equal(raw(got), raw(engine.logits_numpy(two))), step
            assert np.array_equal(raw(got[:, V:]), raw(logits_np[:, V:]))                       # the padding is untouched
            if step % 4 == 0:
                for b in range(n):
                    ref = oms[b].mask(ov)
                    assert np.array_equal(mask_fused[b], ref), (step, b)
                    assert np.array_equal(raw(got[b:b + 1, :V]), raw(O.apply_mask(logits_np[b:b + 1, :V], ref[None, :]))), (step, b)
            toks = [w.trajectories[b][step] for b in range(n)]
            s.accept(toks, restart_on_eos=True)
            for b in range(n):
                if oms[b].accept_token(ov, toks[b]) == 2:
                    oms[b].reset()
        # a terminated request: status XG_ERR_TERMINATED, zero mask row, every logit of its row -inf
        s.reset(0)
        for t in inputs.GreedyTokenizer(w.vocab).encode(w.documents[0][0]) + [w.vocab.eos_id]:
            s.accept([t] + [w.vocab.eos_id] * (n - 1))       # the others refuse end of sequence unless their root is complete
        logits_np = inputs.make_logits(w.logits_seed, n, stride, w.dtype)
        t = engine.logits_tensor(logits_np, s.device)
        s.fill_apply(t)
        assert int(s.status.cpu()[0]) == XG_ERR_TERMINATED and not s.mask_numpy()[0].any()
        got = engine.logits_numpy(t)
        ninf = np.uint32(0xFF800000) if w.dtype == "f32" else np.uint16(0xFF80)
        assert (raw(got[0, :V]) == ninf).all() and np.array_equal(raw(got[0, V:]), raw(logits_np[0, V:]))
    finally:
        s.close()


def test_fill_and_apply_rejects_bad_arguments():
    torch, engine = _engine()
    from paper_2601_04426_b200 import binding as B
    w = inputs.make_workload("C1", steps=2, vocab_size=1024)
    s = engine.Session(w)
    try:
        t = torch.zeros((1, 1024 + 4), dtype=torch.float32, device=s.device)
        for args in [(s.bitmask.data_ptr(), s.W, 0, 0, "f32", 1028), (s.bitmask.data_ptr(), s.W, 0, t.data_ptr(), "f32", 1000),
                     (s.bitmask.data_ptr(), s.W, 0, t.data_ptr() + 4, "f32", 1028), (s.bitmask.data_ptr(), s.W - 1, 0, t.data_ptr(), "f32", 1028),
                     (0, s.W, 0, t.data_ptr(), "f32", 1028)]:
            with pytest.raises(B.XgError) as e:
                s.batch.fill_and_apply_token_bitmask(*args)
            assert e.value.status == B.XG_ERR_INVALID_ARG
    finally:
        s.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_fill_and_apply_with_a_ragged_vocabulary(dtype):
    """A vocabulary that is no multiple of 32 or of the 16-byte vector width: the last word's padding bits and the
    elements behind the last whole vector."""
    torch, engine = _engine()
    from paper_2601_04426_b200 import binding as B
    tokens = [bytes([i]) for i in range(256)] + [b"ab", b"abc.", b"b.", b".", b"zz", b"a.b", b"q" * 9, b"xy", b"."] + [b"pad%d" % i for i in range(11)] + [b""]
    V = len(tokens)
    assert V % 32 and V % 8 and V % 4
    tok = B.Tokenizer(tokens, V - 1)
    g = B.Grammar(tok, "ebnf", 'root ::= [a-z]+ "."')
    m = B.Matcher(g)
    batch = B.Batch([m, m, m])
    ov = O.Vocab(tokens, V - 1)
    om = O.Matcher(O.Grammar('root ::= [a-z]+ "."'))
    W = tok.words
    per16 = 4 if dtype == "f32" else 8
    stride = (V + per16 - 1) // per16 * per16 + per16
    raw = (lambda a: a.view(np.uint32)) if dtype == "f32" else (lambda a: a)
    mask = torch.zeros((3, W), dtype=torch.int32, device="cuda")
    st = torch.zeros(3, dtype=torch.int32, device="cuda")
    ids = torch.zeros(3, dtype=torch.int32, device="cuda")
    for step, t in enumerate([b"ab", b"zz", b"q" * 9, b"."]):
        logits_np = inputs.make_logits(11 + step, 3, stride, dtype)
        lg = engine.logits_tensor(logits_np, "cuda")
        batch.fill_and_apply_token_bitmask(mask.data_ptr(), W, st.data_ptr(), lg.data_ptr(), dtype, stride)
        ref = om.mask(ov)
        got_mask = mask.cpu().numpy().view(np.uint32)
        assert (st.cpu().numpy() == 0).all() and all(np.array_equal(got_mask[r], ref) for r in range(3)), step
        expect = logits_np.copy()
        expect[:, :V] = O.apply_mask(logits_np[:, :V], np.repeat(ref[None, :], 3, axis=0))
        assert np.array_equal(raw(engine.logits_numpy(lg)), raw(expect)), step
        ids[:] = tokens.index(t)
        B.Batch([m]).accept_token(ids.data_ptr(), st.data_ptr())
        assert int(st.cpu()[0]) == 0 and om.accept_token(ov, tokens.index(t)) == 1
    m.close(); g.close(); tok.close()
