"""The allocation-free fill entry point against the regular one (GPU).

Who needs it: a caller that may not allocate device memory inside its decode loop, for instance a
serving engine that gave all free memory to its own allocator, or one that cannot afford the
device-wide synchronisation a cudaMalloc brings.  The regular call creates per-batch device
buffers the first time it sees a batch; the static variant keeps them in a fixed array inside the
library, for at most 1024 requests.  Both must produce the same words.

This file sorts last on purpose: if it fails, `pytest -x` has already run everything else.
"""
import numpy as np
import pytest

from paper_2601_04426_b200 import binding as B
from paper_2601_04426_b200 import inputs

pytestmark = pytest.mark.gpu


def test_static_fill_matches_regular_fill_on_consecutive_calls():
    import torch
    from paper_2601_04426_b200 import engine
    w = inputs.make_workload("C3", batch=6, steps=10, vocab_size=8192)
    s = engine.Session(w)
    try:
        W = s.W
        other = torch.full((s.n, W + 3), -1, dtype=torch.int32, device=s.device)     # padded stride, dirty contents
        other_status = torch.full((s.n,), 77, dtype=torch.int32, device=s.device)
        calls = 0
        for step in range(w.steps):
            s.fill()                                    # regular entry point
            expect = s.bitmask.cpu().numpy()
            expect_status = s.status.cpu().numpy()
            for _ in range(2):                          # two calls in a row share the static array
                other[:, :W] = -1
                s.batch.fill_next_token_bitmask_static(other.data_ptr(), W + 3, other_status.data_ptr(), s.stream())
                got = other.cpu().numpy()
                assert np.array_equal(got[:, :W], expect), step           # integer work: bit for bit
                assert (got[:, W:] == -1).all()                           # nothing written past the row
                assert np.array_equal(other_status.cpu().numpy(), expect_status)
                calls += 1
            toks = [w.trajectories[b][step] for b in range(s.n)]
            s.accept(toks)
            for b in range(s.n):
                if toks[b] == w.vocab.eos_id:
                    s.reset(b)
        assert calls == 2 * w.steps
        # a terminated request: zero row and XG_ERR_TERMINATED from both entry points
        s.reset(0)
        for t in inputs.GreedyTokenizer(w.vocab).encode(w.documents[0][0]) + [w.vocab.eos_id]:
            s.accept([t] * s.n)          # the other requests refuse these tokens and stay where they are
        s.fill()
        expect, expect_status = s.bitmask.cpu().numpy(), s.status.cpu().numpy()
        s.batch.fill_next_token_bitmask_static(other.data_ptr(), W + 3, other_status.data_ptr(), s.stream())
        assert expect_status[0] == B.XG_ERR_TERMINATED and not expect[0].any()
        assert np.array_equal(other.cpu().numpy()[:, :W], expect) and np.array_equal(other_status.cpu().numpy(), expect_status)
    finally:
        s.close()


def test_static_fill_rejects_oversized_batches_and_bad_buffers():
    import torch
    from paper_2601_04426_b200 import engine
    w = inputs.make_workload("C1", steps=2, vocab_size=1024)
    s = engine.Session(w)
    try:
        too_many = B.Batch([s.matchers[0]] * (B.XG_STATIC_FILL_MAX_BATCH + 1))
        big = torch.zeros((4, s.W), dtype=torch.int32, device=s.device)
        with pytest.raises(B.XgError) as e:
            too_many.fill_next_token_bitmask_static(big.data_ptr(), s.W)
        assert e.value.status == B.XG_ERR_CAPACITY and "1024" in str(e.value)
        with pytest.raises(B.XgError) as e:
            s.batch.fill_next_token_bitmask_static(big.data_ptr(), s.W - 1)
        assert e.value.status == B.XG_ERR_INVALID_ARG
        with pytest.raises(B.XgError):
            s.batch.fill_next_token_bitmask_static(0, s.W)
        # the limit itself is accepted (the same request 1024 times: 1024 identical rows)
        full = B.Batch([s.matchers[0]] * B.XG_STATIC_FILL_MAX_BATCH)
        rows = torch.zeros((B.XG_STATIC_FILL_MAX_BATCH, s.W), dtype=torch.int32, device=s.device)
        full.fill_next_token_bitmask_static(rows.data_ptr(), s.W)
        s.fill()
        assert (rows == s.bitmask[0]).all()
    finally:
        s.close()


def test_static_fill_allocates_no_device_memory_where_the_regular_call_does():
    """The property the entry point exists for.  A batch composition that neither call has seen before: the static
    call must leave the device's free memory as it was; the regular call, whose per-batch tables grow on first use
    of a larger batch, serves (with a much larger batch) as the control that the probe would notice an allocation."""
    import torch
    from paper_2601_04426_b200 import engine
    w = inputs.make_workload("C1", steps=2, vocab_size=2048)
    s = engine.Session(w)
    try:
        n_big = 1000
        many = B.Batch([s.matchers[0]] * n_big)
        rows = torch.zeros((n_big, s.W), dtype=torch.int32, device=s.device)
        n_control = 40000                                    # large enough for its tables (tens of MB) to show in the free memory
        control = B.Batch([s.matchers[0]] * n_control)
        rows2 = torch.zeros((n_control, s.W), dtype=torch.int32, device=s.device)
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        many.fill_next_token_bitmask_static(rows.data_ptr(), s.W)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0                                # nothing allocated
        control.fill_next_token_bitmask(rows2.data_ptr(), s.W)      # the regular call grows its per-batch tables here
        torch.cuda.synchronize()
        free2, _ = torch.cuda.mem_get_info()
        assert free2 < free1
        s.fill()
        assert (rows == s.bitmask[0]).all() and (rows2 == s.bitmask[0]).all()
    finally:
        s.close()


def test_static_fill_serves_a_just_in_time_grammar_with_missing_entries():
    """A grammar whose cache entries are not built yet: the static call, like the regular one, takes the mask from a
    walk of the whole vocabulary; both equal the oracle's mask."""
    import torch
    from oracle import oracle as O
    from oracle import schema_ebnf as SE
    w = inputs.make_workload("C1", steps=6, vocab_size=4096)
    v = w.vocab
    tok = B.Tokenizer(v.tokens, v.eos_id, v.special_ids)
    g = B.Grammar(tok, w.grammars[0].kind, w.grammars[0].text, jit=True, jit_precompute=0)
    m = B.Matcher(g)
    batch = B.Batch([m])
    ov = O.Vocab(v.tokens, v.eos_id, v.special_ids)
    om = O.Matcher(O.Grammar(SE.grammar_text(w.grammars[0].kind, w.grammars[0].text)))
    mask = torch.zeros((1, tok.words), dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ids = torch.zeros(1, dtype=torch.int32, device="cuda")
    try:
        for t in w.trajectories[0]:
            for fill in (batch.fill_next_token_bitmask_static, batch.fill_next_token_bitmask):
                mask.fill_(-1)
                fill(mask.data_ptr(), tok.words, st.data_ptr())
                assert int(st.cpu()[0]) == 0 and np.array_equal(mask.cpu().numpy().view(np.uint32)[0], om.mask(ov))
            ids[0] = t
            batch.accept_token(ids.data_ptr(), st.data_ptr())
            if om.accept_token(ov, t) == 2:
                break
    finally:
        m.close(); g.close(); tok.close()
