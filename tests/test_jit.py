"""Just-in-time cache build (Section 3.5) on the GPU: masks stay bit-exact against the oracle
whatever has been built so far, and what gets built equals the full compile's entries."""
import numpy as np
import pytest

from oracle import oracle as O
from oracle import schema_ebnf as SE
from paper_2601_04426_b200 import binding as B
from paper_2601_04426_b200 import inputs

pytestmark = pytest.mark.gpu


def _drive(w, check_every, service, static_fill=False, **session_kw):
    """Run the seeded trajectories with a just-in-time session; compare masks with the oracle."""
    import torch
    from paper_2601_04426_b200 import engine
    s = engine.Session(w, jit=True, **session_kw)
    ov = O.Vocab(w.vocab.tokens, w.vocab.eos_id, w.vocab.special_ids)
    grammars = [O.Grammar(SE.grammar_text(g.kind, g.text)) for g in w.grammars]
    oms = [O.Matcher(grammars[gi]) for gi in w.request_grammar]
    history = []
    try:
        for step in range(w.steps):
            if static_fill:
                s.batch.fill_next_token_bitmask_static(s.bitmask.data_ptr(), s.W, s.status.data_ptr(), s.stream())
            else:
                s.fill()
            mask = s.mask_numpy()
            assert (s.status.cpu().numpy() == 0).all(), step
            toks = [w.trajectories[b][step] for b in range(s.n)]
            for b in range(s.n):
                assert (mask[b, toks[b] >> 5] >> (toks[b] & 31)) & 1, (step, b)
                if step % check_every == 0 or step < 3:
                    ref = oms[b].mask(ov)
                    assert np.array_equal(mask[b], ref), (step, b, int(np.unpackbits((mask[b] ^ ref).view(np.uint8)).sum()))
            s.accept(toks)
            assert (s.accept_status.cpu().numpy() == 0).all(), step
            for b in range(s.n):
                if oms[b].accept_token(ov, toks[b]) == 2:
                    oms[b].reset()
                    s.reset(b)
            if service == "each":
                history.append(s.jit_service(wait=False))
            elif service == "wait":
                history.append(s.jit_service(wait=True))
        final = s.jit_service(wait=True) if service != "never" else s.jit_service(wait=False)
        stats = [g.stats() for g in s.grammars]
        return s, final, history, stats
    except Exception:
        s.close()
        raise


def test_masks_exact_with_nothing_built():
    """No service call at all: every mask comes from the walk of the whole vocabulary."""
    w = inputs.make_workload("C1", steps=40)
    s, final, _, stats = _drive(w, 1, "never")
    assert stats[0]["n_entries_built"] == 0 and final["n_built"] == 0 and final["n_missing"] > 0
    s.close()


def test_masks_exact_while_entries_arrive_between_steps():
    w = inputs.make_workload("C2", steps=120, vocab_size=16384)
    s, final, history, stats = _drive(w, 5, "each")
    assert final["n_built"] > 10 and final["n_in_flight"] == 0
    assert final["n_missing"] > 0, "states the trajectory never visited must stay unbuilt"
    # (C2's repetitions are short: its states do not share entries, every scannable state has its own)
    assert final["n_built"] + final["n_missing"] <= stats[0]["n_scannable"]
    built_so_far = [h["n_built"] for h in history]
    assert built_so_far == sorted(built_so_far) and built_so_far[-1] > built_so_far[2]
    s.close()


def test_built_entries_equal_the_full_compile():
    w = inputs.make_workload("C5", batch=2, steps=60, vocab_size=8192)
    s, final, _, _ = _drive(w, 7, "wait")
    g = s.grammars[0]
    full = B.Grammar(s.tokenizer, w.grammars[0].kind, w.grammars[0].text)
    t = full.tables()
    scannable = [st for st in range(t["n_states"]) if t["cedge_begin"][st + 1] > t["cedge_begin"][st]]
    built = 0
    for st in scannable:
        try:
            e = g.cache_entry(st)
        except B.XgError:
            continue
        built += 1
        ref = full.cache_entry(st)
        assert e["kind"] == ref["kind"] and np.array_equal(e["list"], ref["list"]) and np.array_equal(e["uncertain"], ref["uncertain"]), st
        assert (e["n_accepted"], e["n_uncertain"]) == (ref["n_accepted"], ref["n_uncertain"])
        if e["kind"] == B.XG_STORE_BITSET:
            assert np.array_equal(e["bitset"], ref["bitset"])
    assert built >= final["n_built"] > 0
    full.close(); s.close()


def test_precompute_builds_the_k_costliest_at_compile_time():
    w = inputs.make_workload("C2", steps=2, vocab_size=8192)
    v = w.vocab
    tok = B.Tokenizer(v.tokens, v.eos_id, v.special_ids)
    spec = w.grammars[0]
    full = B.Grammar(tok, spec.kind, spec.text)
    g5 = B.Grammar(tok, spec.kind, spec.text, jit=True, jit_precompute=5)
    gall = B.Grammar(tok, spec.kind, spec.text, jit=True, jit_precompute=10 ** 6)
    assert g5.stats()["n_entries_built"] == 5
    assert gall.stats()["n_entries_built"] == full.stats()["n_entries_built"]
    assert B.jit_service([gall], 0, True)["n_missing"] == 0
    # the five are the ones that leave the fewest tokens to the first-byte test: walking cost = tokens that survive it
    t = full.tables()
    scannable = [st for st in range(t["n_states"]) if t["cedge_begin"][st + 1] > t["cedge_begin"][st]]
    rep = full.state_classes()
    survivors = {}
    for st in scannable:
        if rep[st] != st:
            continue
        e = full.cache_entry(st)
        survivors[st] = e["n_accepted"] + e["n_uncertain"]
    chosen = []
    for st in survivors:
        try:
            g5.cache_entry(st)
            chosen.append(st)
        except B.XgError:
            pass
    assert len(chosen) == 5
    floor = sorted(survivors.values())[-5]
    assert all(survivors[st] * 2 >= floor for st in chosen), (chosen, floor)      # cost is an estimate: same league as the true top five
    for g in (full, g5, gall):
        g.close()
    tok.close()


def test_second_grammar_finds_the_first_ones_entries_in_the_pool():
    import torch
    from paper_2601_04426_b200 import engine
    w = inputs.make_workload("C1", steps=30)
    w2 = inputs.make_workload("C1", steps=30)
    w.grammars = w.grammars + w2.grammars            # the same text twice: two grammars, one pool
    w.request_grammar = [0, 1]
    w.trajectories = [w.trajectories[0], w2.trajectories[0]]
    w.documents = [w.documents[0], w2.documents[0]]
    s = engine.Session(w, jit=True)
    ov = O.Vocab(w.vocab.tokens, w.vocab.eos_id, w.vocab.special_ids)
    om = O.Matcher(O.Grammar(SE.grammar_text(w.grammars[0].kind, w.grammars[0].text)))
    # request 0 walks ahead and gets its entries built; request 1 is fed nothing meanwhile
    first = B.Batch([s.matchers[0]])
    tokens = torch.zeros(1, dtype=torch.int32, device=s.device)
    for step in range(20):
        first.fill_next_token_bitmask(s.bitmask.data_ptr(), s.W, s.status.data_ptr(), s.stream())
        tok = w.trajectories[0][step]
        if tok == w.vocab.eos_id:
            break
        tokens[0] = tok
        first.accept_token(tokens.data_ptr(), s.accept_status.data_ptr(), s.stream())
        B.jit_service([s.grammars[0]], s.stream(), True)
    a = B.jit_service([s.grammars[0]], s.stream(), True)
    assert a["n_built"] > 0 and a["n_pool_hits"] == 0
    second = B.Batch([s.matchers[1]])
    for step in range(20):
        second.fill_next_token_bitmask(s.bitmask.data_ptr(), s.W, s.status.data_ptr(), s.stream())
        assert np.array_equal(s.mask_numpy()[0], om.mask(ov)), step
        tok = w.trajectories[1][step]
        if tok == w.vocab.eos_id:
            break
        tokens[0] = tok
        second.accept_token(tokens.data_ptr(), s.accept_status.data_ptr(), s.stream())
        om.accept_token(ov, tok)
        B.jit_service([s.grammars[1]], s.stream(), True)
    b = B.jit_service([s.grammars[1]], s.stream(), True)
    assert b["n_pool_hits"] > 0 and b["n_built"] == 0
    s.close()


def test_allocation_free_fill_and_many_grammars():
    """The two-kernel fill path takes the same fallback; a batch of grammars shares one pool."""
    w = inputs.make_workload("C3", batch=6, steps=40, vocab_size=8192)
    s, final, _, _ = _drive(w, 6, "each", static_fill=True)
    assert final["n_built"] + final["n_pool_hits"] > 0
    s.close()


def test_arena_that_is_too_small_is_replaced_by_a_larger_one():
    """Builds that find no room in the pool's just-in-time arena are repeated in a larger arena;
    the masks are exact meanwhile and afterwards."""
    w = inputs.make_workload("C1", steps=50)
    s, final, _, _ = _drive(w, 2, "wait", jit_arena_bytes=4096)
    assert final["n_built"] > 0 and final["n_in_flight"] == 0
    pool = s.pool.stats()
    assert pool["chunks"] >= 2                   # the first arena (4 KiB) and at least one successor
    s.close()


def test_long_tokens_take_the_exact_build_path():
    """A vocabulary with tokens beyond the fast path's 32 bytes: the just-in-time build notices on the
    device that it cannot finish, and the service call falls back to the exact build."""
    import torch
    base = [bytes([b]) for b in range(256)]
    long_tokens = [b"a" * 33, b"ab" * 40, b"x" * 255, b"a" * 40 + b"}", b"a" * 100 + b"}}", b"b" * 64 + b'}, "k": {', b'{"' + b"q" * 60]
    toks = base + long_tokens + [b""]
    toks += [b"\xfe\xff%d" % i for i in range(-len(toks) % 32)]
    eos = toks.index(b"")
    ebnf = 'root ::= obj\nobj ::= "{" [a-z]* "}" | "{" "\\"" [a-z]* "\\": " obj "}"\n'
    tok = B.Tokenizer(toks, eos)
    g = B.Grammar(tok, "ebnf", ebnf, inline_max_states=0, jit=True)
    full = B.Grammar(tok, "ebnf", ebnf, inline_max_states=0)
    ov = O.Vocab(toks, eos)
    om = O.Matcher(O.Grammar(ebnf))
    m = B.Matcher(g)
    batch = B.Batch([m])
    mask = torch.zeros((1, tok.words), dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ids = torch.zeros(1, dtype=torch.int32, device="cuda")
    for piece in [b"{", b'"', b"q", b"q", b'"', b":", b" ", b"{", b"a" * 33, b"ab" * 40, b"a" * 40 + b"}", b"}"]:
        for _ in range(2):                       # once from the whole-vocabulary walk, once more after the service call
            batch.fill_next_token_bitmask(mask.data_ptr(), tok.words, st.data_ptr())
            assert int(st.cpu()[0]) == 0
            assert np.array_equal(mask.cpu().numpy().view(np.uint32)[0], om.mask(ov)), piece
            B.jit_service([g], 0, True)
            m2 = B.Matcher(g)                    # a fresh matcher fed the same bytes sees the published entries
            m2.close()
        tid = toks.index(piece)
        ids[0] = tid
        batch.accept_token(ids.data_ptr(), st.data_ptr())
        assert int(st.cpu()[0]) == 0, piece
        assert om.accept_token(ov, tid) == 1
    stats = B.jit_service([g], 0, True)
    assert stats["n_built"] > 0
    t = full.tables()
    compared = 0
    for s_ in [x for x in range(t["n_states"]) if t["cedge_begin"][x + 1] > t["cedge_begin"][x]]:
        try:
            e = g.cache_entry(s_)
        except B.XgError:
            continue
        ref = full.cache_entry(s_)
        assert e["kind"] == ref["kind"] and np.array_equal(e["list"], ref["list"]) and np.array_equal(e["uncertain"], ref["uncertain"]), s_
        compared += 1
    assert compared > 0
    m.close(); g.close(); full.close(); tok.close()


def test_teardown_with_builds_in_flight_and_pool_accounting():
    import torch
    from paper_2601_04426_b200 import engine
    w = inputs.make_workload("C3", batch=4, steps=12, vocab_size=8192)
    s = engine.Session(w, jit=True)
    for step in range(6):
        s.fill()
        s.accept([w.trajectories[b][step] for b in range(s.n)])
        s.jit_service(wait=False)                # leaves a snapshot or builds on their way
    pool, tokenizer = s.pool, s.tokenizer
    before = pool.stats()
    assert before["bytes"] > 0
    pool.set_limit(1)                            # everything held is in use by the live grammars
    assert pool.stats()["evicted_chunks"] == 0
    for m in s.matchers:                         # matchers and grammars go while work may be pending
        m.close()
    for g in s.grammars:
        g.close()
    after = pool.stats()
    assert after["bytes"] == 0 and after["chunks"] == 0
    # the pool is still usable: a new just-in-time grammar starts from nothing
    g = B.Grammar(tokenizer, w.grammars[0].kind, w.grammars[0].text, pool=pool, jit=True, jit_precompute=3)
    assert g.stats()["n_entries_built"] == 3
    g.close()
    pool.close(); tokenizer.close()


def test_just_in_time_entries_serve_whole_classes_of_states():
    """Long repetitions: one entry built just in time is published to every state of its class
    (repetition state compression), so a string of hundreds of characters costs a handful of builds."""
    w = inputs.make_workload("R256", batch=4, steps=150, vocab_size=8192)
    s, final, _, stats = _drive(w, 6, "each", repeat_threshold=-1)
    assert 0 < final["n_built"] < 400
    assert sum(x["n_states"] for x in stats) > 20 * final["n_built"]
    s.close()
