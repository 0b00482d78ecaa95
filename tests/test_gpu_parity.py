"""GPU parity: every bitmask word, cache entry and masked logit against the CPU oracle.

All calls go through the C ABI (via the ctypes binding).  Integer work is compared bit for bit.
"""
import json

import numpy as np
import pytest

from oracle import oracle as O
from oracle import schema_ebnf as SE
from paper_2601_04426_b200 import binding as B
from paper_2601_04426_b200 import inputs

pytestmark = pytest.mark.gpu


def _engine():
    import torch
    from paper_2601_04426_b200 import engine
    return torch, engine


def _oracle_side(w):
    ov = O.Vocab(w.vocab.tokens, w.vocab.eos_id, w.vocab.special_ids)
    grammars = [O.Grammar(SE.grammar_text(g.kind, g.text)) for g in w.grammars]
    matchers = [O.Matcher(grammars[gi]) for gi in w.request_grammar]
    return ov, grammars, matchers


def _run_trajectories(w, check_steps, check_requests=None, fused=False, restart=False, **session_kw):
    """Drive GPU and oracle along the seeded trajectories; compare masks where asked, and the
    cheap invariants everywhere (sampled token allowed, statuses, termination).  fused: after the
    first fill every step is one accept-and-fill launch that restarts a request at end of
    sequence, instead of accept, reset and fill.  restart: the accept call restarts a request at
    end of sequence (no reset call)."""
    torch, engine = _engine()
    s = engine.Session(w, **session_kw)
    ov, _, oms = _oracle_side(w)
    n = s.n
    compared = 0
    try:
        for step in range(w.steps):
            if step == 0 or not fused:
                s.fill()
            mask = s.mask_numpy()
            status = s.status.cpu().numpy()
            assert (status == 0).all(), (step, status)
            toks = [w.trajectories[b][step] for b in range(n)]
            for b in range(n):
                assert (mask[b, toks[b] >> 5] >> (toks[b] & 31)) & 1, (step, b, w.vocab.tokens[toks[b]])
                if step in check_steps or (check_requests is not None and b in check_requests):
                    ref = oms[b].mask(ov)
                    if not np.array_equal(mask[b], ref):
                        diff = np.nonzero(O.unpack_bits(mask[b] ^ ref, ov.size))[0]
                        raise AssertionError("step %d request %d: %d differing tokens, e.g. %r (gpu=%d)" % (
                            step, b, len(diff), [w.vocab.tokens[t] for t in diff[:8]], int((mask[b, diff[0] >> 5] >> (diff[0] & 31)) & 1)))
                    compared += 1
            if fused:
                s.accept_fill(toks, restart_on_eos=True)
            else:
                s.accept(toks, restart_on_eos=restart)
            ast = s.accept_status.cpu().numpy()
            assert (ast == 0).all(), (step, ast)
            for b in range(n):
                r = oms[b].accept_token(ov, toks[b])
                assert r in (1, 2)
                if r == 2:
                    assert s.matchers[b].is_terminated() != (fused or restart)
                    oms[b].reset()
                    if not (fused or restart):
                        s.reset(b)
        return compared
    finally:
        s.close()


def test_c1_every_step_bit_exact():
    w = inputs.make_workload("C1")
    assert _run_trajectories(w, set(range(w.steps))) == w.steps


def test_c2_sampled_steps_bit_exact():
    w = inputs.make_workload("C2", steps=96)
    assert _run_trajectories(w, set(range(0, 96, 4))) == 24


def test_c3_inter_request_batch():
    w = inputs.make_workload("C3", batch=16, steps=48)
    _run_trajectories(w, {0, 5, 17, 33, 47}, check_requests={3})


def test_c4_tag_dispatch_batch():
    w = inputs.make_workload("C4", batch=6, steps=120)
    _run_trajectories(w, {0, 1, 30, 60, 119}, check_requests={2})


def test_c5_recursive_json_with_utf8():
    w = inputs.make_workload("C5", batch=8, steps=64)
    _run_trajectories(w, {0, 7, 31, 63}, check_requests={1})


def test_many_tag_dispatch_batch():
    """Twenty tags with a common prefix (the paper's tag-count experiment, Section 4.1)."""
    w = inputs.make_workload("T20", batch=4, steps=90, vocab_size=16384)
    _run_trajectories(w, {0, 20, 45, 89}, check_requests={1})


def test_channel_protocol_batch():
    """Text channels that run to a stop string, tool channels, a final stop string (Sections 1, 3.2)."""
    w = inputs.make_workload("H16", batch=6, steps=140, vocab_size=16384)
    _run_trajectories(w, {0, 1, 15, 40, 80, 139}, check_requests={4})


def test_hand_worked_masks_on_gpu():
    torch, engine = _engine()
    from golden_util import load_mask_fixture
    for fixture in ["mask_ab_ac.txt", "mask_bool_object.txt", "mask_nested_arrays.txt"]:
        ebnf, tokens, cases = load_mask_fixture(fixture)
        toks = [t.encode() for t in tokens]
        eos = tokens.index("")
        feed = toks + [bytes([b]) for b in range(256)]         # extra single bytes, only used to feed prefixes
        feed += [b"\xff\xfe"] * (-len(feed) % 32)
        tok = B.Tokenizer(feed, eos)
        g = B.Grammar(tok, "ebnf", ebnf)
        m = B.Matcher(g)
        batch = B.Batch([m])
        words = tok.words
        mask = torch.zeros((1, words), dtype=torch.int32, device="cuda")
        ids = torch.zeros(1, dtype=torch.int32, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        for prefix, allowed in cases:
            m.reset()
            rest = prefix.encode()
            while rest:                          # feed the prefix with the longest tokens available
                cand = max((t for t in feed if t and rest.startswith(t)), key=len)
                ids[0] = feed.index(cand)
                batch.accept_token(ids.data_ptr(), st.data_ptr())
                assert int(st.cpu()[0]) == 0, (prefix, cand)
                rest = rest[len(cand):]
            batch.fill_next_token_bitmask(mask.data_ptr(), words, st.data_ptr())
            bits = O.unpack_bits(mask.cpu().numpy().view(np.uint32)[0], len(tokens))
            got = sorted(tokens[i] for i in range(len(tokens)) if bits[i])
            assert got == sorted(allowed), (fixture, prefix, got)
        m.close(); g.close(); tok.close()


def _entry_sets(entry, V):
    unc = set(entry["uncertain"].tolist())
    if entry["kind"] == B.XG_STORE_ACCEPT_LIST:
        acc = set(entry["list"].tolist())
    elif entry["kind"] == B.XG_STORE_REJECT_LIST:
        acc = set(range(V)) - set(entry["list"].tolist()) - unc
    else:
        acc = set(np.nonzero(O.unpack_bits(entry["bitset"], V))[0].tolist())
    return acc, unc


def test_hand_worked_classification_on_gpu():
    """The cache entries of a two-rule grammar against the table worked out on paper from Section 3.4."""
    from golden_util import load_classify_fixture, state_at_path
    ebnf, tokens, cases = load_classify_fixture("classify_bracket_item.txt")
    tok = B.Tokenizer([t.encode() for t in tokens], tokens.index(""))
    g = B.Grammar(tok, "ebnf", ebnf, inline_max_states=0)
    t = g.tables()
    for path, acc, unc in cases:
        e = g.cache_entry(state_at_path(t, path))
        got_acc, got_unc = _entry_sets(e, len(tokens))
        assert sorted(tokens[i] for i in got_acc) == sorted(acc), path
        assert sorted(tokens[i] for i in got_unc) == sorted(unc), path
    g.close(); tok.close()


def _entry_classes(entry, V):
    """uint8[V] in the oracle's coding (1 accepted, 2 uncertain, 0 rejected) from a cache entry view."""
    cls = np.zeros(V, dtype=np.uint8)
    unc = entry["uncertain"]
    if entry["kind"] == B.XG_STORE_ACCEPT_LIST:
        cls[entry["list"]] = 1
    elif entry["kind"] == B.XG_STORE_REJECT_LIST:
        cls[:] = 1
        cls[entry["list"]] = 0
    else:
        cls[O.unpack_bits(entry["bitset"], V)] = 1
    assert not cls[unc].any() or entry["kind"] == B.XG_STORE_REJECT_LIST      # uncertain ids are outside the stored accepted set
    cls[unc] = 2
    return cls


def _oracle_tables(g):
    t = g.tables()
    scal = {k: t.pop(k) for k in ("n_rules", "n_states", "n_classes", "root_rule", "root_nullable")}
    return O.Tables(scal["n_rules"], scal["n_states"], scal["n_classes"], scal["root_rule"], scal["root_nullable"], **t), t


def _check_entry(g, tb, ov, s, words):
    """One cache entry against the oracle's classification row of its state: the three sets, list
    order, counts, and that the stored form is the smallest (ties: accepted list, rejected list, bitset)."""
    e = g.cache_entry(s)
    V = ov.size
    ref = tb.classify(ov, s)
    got = _entry_classes(e, V)
    if not np.array_equal(got, ref):
        bad = np.nonzero(got != ref)[0]
        raise AssertionError("state %d: %d tokens differ, e.g. %r (library %d, oracle %d)" % (s, len(bad), ov.tokens[bad[0]], got[bad[0]], ref[bad[0]]))
    assert (np.diff(e["uncertain"]) > 0).all() and (np.diff(e["list"]) > 0).all()
    n_acc, n_unc = int((ref == 1).sum()), int((ref == 2).sum())
    n_rej = V - n_acc - n_unc
    assert (e["n_accepted"], e["n_uncertain"], e["n_rejected"]) == (n_acc, n_unc, n_rej)
    sizes = [4 * n_acc, 4 * n_rej, 4 * words]
    assert e["kind"] == sizes.index(min(sizes)), (s, sizes, e["kind"])
    return e["kind"]


def _seeded_sample(states, share, seed):
    """A seeded `share` of `states` (at least one), in ascending order."""
    rng = inputs.Rng(seed)
    k = max(1, int(round(len(states) * share)))
    pool = list(states)
    picked = []
    for _ in range(min(k, len(pool))):
        picked.append(pool.pop(rng.below(len(pool))))
    return sorted(picked)


# Cache parity at the full vocabulary of each config: every scannable state for C1 and C5, a seeded
# 5 % of the states (the whole vocabulary each) for C2 and C4; C3 has a test of its own below.
@pytest.mark.parametrize("name,share", [("C1", 1.0), ("C5", 1.0), ("C2", 0.05), ("C4", 0.05)])
def test_cache_entries_match_oracle_classification(name, share):
    torch, engine = _engine()
    w = inputs.make_workload(name, batch=1, steps=2)
    v = w.vocab
    tok = B.Tokenizer(v.tokens, v.eos_id, v.special_ids)
    g = B.Grammar(tok, w.grammars[0].kind, w.grammars[0].text)
    tb, t = _oracle_tables(g)
    ov = O.Vocab(v.tokens, v.eos_id, v.special_ids)
    states = tb.scannable_states()
    stats = g.stats()
    assert stats["n_scannable"] == len(states)
    picked = states if share >= 1.0 else _seeded_sample(states, share, inputs.config_seed(name) ^ 0xCAC4E)
    kinds = {_check_entry(g, tb, ov, s, tok.words) for s in picked}
    if name == "C5":
        assert B.XG_STORE_ACCEPT_LIST in kinds and B.XG_STORE_BITSET in kinds
        # the grammar's lookahead drops uncertain tokens whose next byte can follow their rule nowhere
        assert 0 < stats["total_checked"] < stats["total_uncertain"]
    if name == "C4":
        # free text accepts nearly everything: the root automaton's start state stores a rejected list
        assert _check_entry(g, tb, ov, int(t["rule_start"][0]), tok.words) == B.XG_STORE_REJECT_LIST
    g.close(); tok.close()


def test_cache_entries_of_all_c3_grammars_match_oracle_classification():
    """C3 as the benchmark compiles it: 128 grammars into one pool from several host threads, so most entries
    come from another grammar's build.  A seeded 5 % of every grammar's scannable states, whole vocabulary each."""
    torch, engine = _engine()
    w = inputs.make_workload("C3", steps=2)
    s = engine.Session(w)
    ov = O.Vocab(w.vocab.tokens, w.vocab.eos_id, w.vocab.special_ids)
    checked = 0
    try:
        for gi, g in enumerate(s.grammars):
            tb, _ = _oracle_tables(g)
            for st in _seeded_sample(tb.scannable_states(), 0.05, inputs.config_seed("C3") ^ (0xCAC4E + gi)):
                _check_entry(g, tb, ov, st, s.W)
                checked += 1
        assert checked >= 0.04 * sum(g.stats()["n_scannable"] for g in s.grammars)
    finally:
        s.close()


def test_cross_grammar_pool_reuses_entries():
    torch, engine = _engine()
    w = inputs.make_workload("C3", batch=6, steps=2, vocab_size=4096)
    v = w.vocab
    tok = B.Tokenizer(v.tokens, v.eos_id, v.special_ids)
    pool = B.CachePool(tok)
    shared = [B.Grammar(tok, g.kind, g.text, pool=pool) for g in w.grammars]
    private = [B.Grammar(tok, g.kind, g.text) for g in w.grammars]
    reused = sum(g.stats()["n_entries_reused"] for g in shared)
    assert reused > 0 and shared[0].stats()["n_entries_reused"] >= 0
    assert sum(g.stats()["n_entries_built"] for g in shared) < sum(g.stats()["n_entries_built"] for g in private)
    # the same text compiled twice into one pool builds nothing the second time
    again = B.Grammar(tok, w.grammars[0].kind, w.grammars[0].text, pool=pool)
    assert again.stats()["n_entries_built"] == 0
    for a, b in zip(shared, private):           # reuse never changes an entry
        t = a.tables()
        scannable = [s for s in range(t["n_states"]) if t["cedge_begin"][s + 1] > t["cedge_begin"][s]]
        for s in scannable[::29]:
            ea, eb = a.cache_entry(s), b.cache_entry(s)
            assert ea["kind"] == eb["kind"] and np.array_equal(ea["list"], eb["list"]) and np.array_equal(ea["uncertain"], eb["uncertain"])
    for g in shared + private + [again]:
        g.close()
    pool.close(); tok.close()


def _scannable(g):
    t = g.tables()
    return [s for s in range(t["n_states"]) if t["cedge_begin"][s + 1] > t["cedge_begin"][s]]


def _same_entries(a, b, stride=1):
    for s in _scannable(a)[::stride]:
        ea, eb = a.cache_entry(s), b.cache_entry(s)
        assert ea["kind"] == eb["kind"] and np.array_equal(ea["list"], eb["list"]) and np.array_equal(ea["uncertain"], eb["uncertain"]), s


def test_pool_limit_never_evicts_entries_in_use():
    """Section 3.3: the pool has a size limit; eviction must not touch what a live grammar reads."""
    torch, engine = _engine()
    w = inputs.make_workload("C3", batch=4, steps=2, vocab_size=4096)
    v = w.vocab
    tok = B.Tokenizer(v.tokens, v.eos_id, v.special_ids)
    pool = B.CachePool(tok)
    shared = [B.Grammar(tok, g.kind, g.text, pool=pool) for g in w.grammars]
    private = [B.Grammar(tok, g.kind, g.text) for g in w.grammars]
    before = pool.stats()
    assert before["bytes"] > 0 and before["evicted_chunks"] == 0 and before["live_rules"] > 0
    assert before["reserved_bytes"] >= before["bytes"]
    pool.set_limit(1)                           # far below what is held, but all of it is in use
    assert pool.stats() == before
    last = shared.pop()
    last.close()                                # what only this grammar used may go now
    after = pool.stats()
    assert after["evicted_chunks"] >= 1 and after["bytes"] < before["bytes"] and after["live_rules"] < before["live_rules"]
    assert after["bytes"] + after["evicted_bytes"] == before["bytes"]
    for a, b in zip(shared, private):           # the survivors still read valid memory
        _same_entries(a, b, stride=17)
    # the evicted rules are rebuilt on demand, with the same result
    again = B.Grammar(tok, w.grammars[3].kind, w.grammars[3].text, pool=pool)
    assert again.stats()["n_entries_built"] > 0
    _same_entries(again, private[3], stride=7)
    for g in shared + private + [again]:
        g.close()
    assert pool.stats()["bytes"] == 0 and pool.stats()["chunks"] == 0 and pool.stats()["reserved_bytes"] == 0
    pool.close(); tok.close()


def test_pool_evicts_in_least_recently_used_order():
    torch, engine = _engine()
    w = inputs.make_workload("C1", batch=1, steps=2, vocab_size=4096)
    v = w.vocab
    tok = B.Tokenizer(v.tokens, v.eos_id, v.special_ids)
    pool = B.CachePool(tok)
    texts = {k: 'root ::= "%s"+ [0-9]' % k for k in "abc"}

    def compile_and_drop(k):
        g = B.Grammar(tok, "ebnf", texts[k], pool=pool)
        built = g.stats()["n_entries_built"]
        g.close()
        return built

    assert all(compile_and_drop(k) > 0 for k in "abc")       # use order: a, b, c
    assert compile_and_drop("a") == 0                        # now: b, c, a
    s = pool.stats()
    assert s["chunks"] == 3 and s["evicted_chunks"] == 0
    pool.set_limit(s["bytes"] - 1)                           # one batch of entries has to go: b's
    s = pool.stats()
    assert s["chunks"] == 2 and s["evicted_chunks"] == 1
    assert compile_and_drop("a") == 0 and compile_and_drop("c") == 0
    assert compile_and_drop("b") > 0                         # rebuilt; to stay under the limit the oldest idle one (a) went
    assert pool.stats()["evicted_chunks"] == 2
    assert compile_and_drop("c") == 0 and compile_and_drop("a") > 0
    pool.set_limit(0)                                        # no limit again: nothing more is evicted
    n = pool.stats()["evicted_chunks"]
    assert compile_and_drop("b") >= 0 and compile_and_drop("c") >= 0 and pool.stats()["evicted_chunks"] == n
    pool.close(); tok.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("rows,vocab,stride_pad", [(1, 8192, 0), (3, 1000, 8), (5, 32 * 7 + 5, 16), (2, 151936, 0)])
def test_apply_matches_oracle(dtype, rows, vocab, stride_pad):
    torch, engine = _engine()
    elt_per_16 = 4 if dtype == "f32" else 8
    stride = ((vocab + elt_per_16 - 1) // elt_per_16) * elt_per_16 + stride_pad
    full = inputs.make_logits(5, rows, stride, dtype)
    if dtype == "f32":
        full[0, 3] = np.nan; full[0, 4] = -0.0; full[rows - 1, vocab - 1] = np.inf
    else:
        full[0, 3] = 0x7FC1; full[0, 4] = 0x8000; full[rows - 1, vocab - 1] = 0x7F80
    words = (vocab + 31) // 32
    mstride = words + 3
    bits = (inputs.stream_u64(9, rows * mstride * 32).reshape(rows, mstride * 32) % 5) < 2
    bits[0, :64] = True            # an all-allowed vector group
    bits[0, 64:160] = False        # an all-masked group
    bits[0, 3] = False
    mask = np.packbits(bits.astype(np.uint8), axis=1, bitorder="little").view(np.uint32).reshape(rows, mstride)
    expect = full.copy()
    expect[:, :vocab] = O.apply_mask(full[:, :vocab], mask[:, :words])
    t = engine.logits_tensor(full, "cuda")
    dmask = torch.from_numpy(mask.view(np.int32)).cuda()
    B.apply_token_bitmask(t.data_ptr(), dtype, rows, vocab, stride, dmask.data_ptr(), mstride)
    got = engine.logits_numpy(t)
    raw = (lambda a: a.view(np.uint32)) if dtype == "f32" else (lambda a: a)
    assert np.array_equal(raw(got), raw(expect))
    # a subset of rows through row_indices leaves the others untouched
    if rows >= 3:
        t2 = engine.logits_tensor(full, "cuda")
        idx = torch.tensor([2, 0], dtype=torch.int32, device="cuda")
        B.apply_token_bitmask(t2.data_ptr(), dtype, rows, vocab, stride, dmask.data_ptr(), mstride, idx.data_ptr(), 2)
        got2 = engine.logits_numpy(t2)
        assert np.array_equal(raw(got2[[0, 2]]), raw(expect[[0, 2]])) and np.array_equal(raw(got2[1]), raw(full[1]))


def test_apply_rejects_bad_arguments():
    torch, engine = _engine()
    t = torch.zeros((2, 64), dtype=torch.float32, device="cuda")
    m = torch.zeros((2, 2), dtype=torch.int32, device="cuda")
    for args in [(0, "f32", 2, 64, 64, m.data_ptr(), 2), (t.data_ptr(), "f32", 2, 64, 32, m.data_ptr(), 2),
                 (t.data_ptr(), "f32", 2, 64, 64, m.data_ptr(), 1), (t.data_ptr() + 4, "f32", 2, 60, 64, m.data_ptr(), 2)]:
        with pytest.raises(B.XgError) as e:
            B.apply_token_bitmask(*args)
        assert e.value.status == B.XG_ERR_INVALID_ARG


def test_statuses_rejected_terminated_and_mixed_grammars():
    torch, engine = _engine()
    toks = [bytes([b]) for b in range(256)] + [b"ab", b"abc", b"true", b"", b"<sp>"] + [b"zz%d" % i for i in range(27)]
    eos = toks.index(b"")
    tok = B.Tokenizer(toks, eos, [toks.index(b"<sp>")])
    g1 = B.Grammar(tok, "ebnf", 'root ::= "ab" "c"?')
    g2 = B.Grammar(tok, "json_schema", json.dumps({"type": "boolean"}))
    g3 = B.Grammar(tok, "ebnf", 'root ::= ""')                      # only the empty string
    ms = [B.Matcher(g1), B.Matcher(g2), B.Matcher(g3)]
    batch = B.Batch(ms)
    W = tok.words
    mask = torch.zeros((3, W + 2), dtype=torch.int32, device="cuda")
    st = torch.zeros(3, dtype=torch.int32, device="cuda")
    ids = torch.zeros(3, dtype=torch.int32, device="cuda")

    def allowed(row):
        bits = O.unpack_bits(mask.cpu().numpy().view(np.uint32)[row, :W], len(toks))
        return sorted(toks[i] for i in np.nonzero(bits)[0])

    batch.fill_next_token_bitmask(mask.data_ptr(), W + 2, st.data_ptr())
    assert allowed(0) == sorted([b"a", b"ab", b"abc"]) and allowed(1) == sorted([b"t", b"f", b"true"]) and allowed(2) == [b""]
    assert st.cpu().tolist() == [0, 0, 0]
    # request 0 takes "ab"; request 1 tries a refused token; request 2 ends
    ids.copy_(torch.tensor([toks.index(b"ab"), toks.index(b"x"), eos], dtype=torch.int32))
    batch.accept_token(ids.data_ptr(), st.data_ptr())
    assert st.cpu().tolist() == [0, B.XG_ERR_TOKEN_REJECTED, 0]
    assert ms[2].is_terminated() and not ms[1].is_terminated()
    batch.fill_next_token_bitmask(mask.data_ptr(), W + 2, st.data_ptr())
    assert allowed(0) == sorted([b"c", b""]) and allowed(1) == sorted([b"t", b"f", b"true"]) and allowed(2) == []
    assert st.cpu().tolist() == [0, 0, B.XG_ERR_TERMINATED]
    # special token, EOS too early, out-of-range id
    ids.copy_(torch.tensor([toks.index(b"<sp>"), eos, 10 ** 6], dtype=torch.int32))
    batch.accept_token(ids.data_ptr(), st.data_ptr())
    assert st.cpu().tolist() == [B.XG_ERR_TOKEN_REJECTED, B.XG_ERR_TOKEN_REJECTED, B.XG_ERR_TERMINATED]
    ms[2].reset()
    batch.fill_next_token_bitmask(mask.data_ptr(), W + 2, st.data_ptr())
    assert allowed(2) == [b""] and st.cpu().tolist() == [0, 0, 0]
    with pytest.raises(B.XgError):
        batch.fill_next_token_bitmask(mask.data_ptr(), W - 1, st.data_ptr())
    for m in ms:
        m.close()
    for g in (g1, g2, g3):
        g.close()
    tok.close()


def test_history_capacity_is_reported_not_overrun():
    torch, engine = _engine()
    toks = [bytes([b]) for b in range(256)] + [b"aaaa", b""] + [b"pad%d" % i for i in range(30)]
    eos = toks.index(b"")
    tok = B.Tokenizer(toks, eos)
    g = B.Grammar(tok, "ebnf", 'root ::= "a"*')
    m = B.Matcher(g, max_sets=10)
    batch = B.Batch([m])
    ids = torch.tensor([toks.index(b"aaaa")], dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    seen = []
    for _ in range(4):
        batch.accept_token(ids.data_ptr(), st.data_ptr())
        seen.append(int(st.cpu()[0]))
    assert seen == [0, 0, B.XG_ERR_CAPACITY, B.XG_ERR_CAPACITY]
    mask = torch.zeros((1, tok.words), dtype=torch.int32, device="cuda")
    batch.fill_next_token_bitmask(mask.data_ptr(), tok.words, st.data_ptr())       # state still usable
    bits = O.unpack_bits(mask.cpu().numpy().view(np.uint32)[0], len(toks))
    assert bits[ord("a")] and bits[eos] and bits[toks.index(b"aaaa")] and bits.sum() == 3
    m.close(); g.close(); tok.close()


def test_long_tokens_up_to_255_bytes():
    """Tokens beyond the per-thread walk arrays (33..255 bytes): classified by the exact slow path at
    build time, accepted in pieces, and checked against the full state when uncertain."""
    torch, engine = _engine()
    base = [bytes([b]) for b in range(256)]
    long_tokens = [b"a" * 33, b"ab" * 40, b"x" * 255, b"a" * 40 + b"}", b"a" * 100 + b"}}", b"b" * 64 + b'}, "k": {', b"z" * 200 + b"}!", b'{"' + b"q" * 60]
    toks = base + long_tokens + [b""]
    toks += [b"\xfe\xff%d" % i for i in range(-len(toks) % 32)]
    eos = toks.index(b"")
    ebnf = 'root ::= obj\nobj ::= "{" [a-z]* "}" | "{" "\\"" [a-z]* "\\": " obj "}"\n'
    tok = B.Tokenizer(toks, eos)
    g = B.Grammar(tok, "ebnf", ebnf, inline_max_states=0)
    ov = O.Vocab(toks, eos)
    og = O.Grammar(ebnf)
    # cache entries against the oracle's classification on the exported tables
    t = g.tables()
    scal = {k: t.pop(k) for k in ("n_rules", "n_states", "n_classes", "root_rule", "root_nullable")}
    tb = O.Tables(scal["n_rules"], scal["n_states"], scal["n_classes"], scal["root_rule"], scal["root_nullable"], **t)
    saw_long_uncertain = False
    for s_ in tb.scannable_states():
        e = g.cache_entry(s_)
        cls = tb.classify(ov, s_)
        acc, unc = _entry_sets(e, len(toks))
        assert acc == set(np.nonzero(cls == 1)[0].tolist()) and unc == set(np.nonzero(cls == 2)[0].tolist()), s_
        saw_long_uncertain |= any(len(toks[i]) > 32 for i in unc)
    assert saw_long_uncertain
    m = B.Matcher(g)
    batch = B.Batch([m])
    om = O.Matcher(og)
    mask = torch.zeros((1, tok.words), dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ids = torch.zeros(1, dtype=torch.int32, device="cuda")
    for piece in [b"{", b'"', b"q" * 3, b'": ', b"{", b"a" * 33, b"ab" * 40, b"a" * 40 + b"}", b"}"]:
        batch.fill_next_token_bitmask(mask.data_ptr(), tok.words, st.data_ptr())
        assert int(st.cpu()[0]) == 0
        assert np.array_equal(mask.cpu().numpy().view(np.uint32)[0], om.mask(ov)), piece
        tid = toks.index(piece) if piece in toks else None
        if tid is None:
            for byte in piece:
                ids[0] = byte
                batch.accept_token(ids.data_ptr(), st.data_ptr())
                assert int(st.cpu()[0]) == 0
                assert om.accept_token(ov, byte) == 1
        else:
            ids[0] = tid
            batch.accept_token(ids.data_ptr(), st.data_ptr())
            assert int(st.cpu()[0]) == 0, piece
            assert om.accept_token(ov, tid) == 1
    batch.fill_next_token_bitmask(mask.data_ptr(), tok.words, st.data_ptr())
    assert np.array_equal(mask.cpu().numpy().view(np.uint32)[0], om.mask(ov))
    m.close(); g.close(); tok.close()
    # the same through the two-kernel fill of the allocation-free entry point, and with a just-in-time grammar whose
    # entries are all missing (the whole vocabulary, long tokens included, is walked against the Earley state)
    feed = [b"{", b'"', b"q", b"q", b'"', b":", b" ", b"{", b"a" * 33, b"ab" * 40, b"a" * 40 + b"}", b"}"]
    _drive(ebnf, toks, eos, feed, static_too=True)
    tok = B.Tokenizer(toks, eos)
    gj = B.Grammar(tok, "ebnf", ebnf, inline_max_states=0, jit=True, jit_precompute=0)
    mj = B.Matcher(gj)
    bj = B.Batch([mj])
    om = O.Matcher(og)
    for piece in feed:
        for fill in (bj.fill_next_token_bitmask, bj.fill_next_token_bitmask_static):
            fill(mask.data_ptr(), tok.words, st.data_ptr())
            assert int(st.cpu()[0]) == 0 and np.array_equal(mask.cpu().numpy().view(np.uint32)[0], om.mask(ov)), piece
        ids[0] = toks.index(piece)
        bj.accept_token(ids.data_ptr(), st.data_ptr())
        assert int(st.cpu()[0]) == 0 and om.accept_token(ov, toks.index(piece)) == 1
    mj.close(); gj.close(); tok.close()


def _drive(ebnf, toks, eos, feed, inline=0, static_too=False):
    """Feed `feed` (token byte strings) to a matcher of grammar `ebnf`, comparing every mask (and the static
    entry point's, when asked) and every accept status with the oracle."""
    torch, engine = _engine()
    tok = B.Tokenizer(toks, eos)
    g = B.Grammar(tok, "ebnf", ebnf, inline_max_states=inline)
    ov = O.Vocab(toks, eos)
    om = O.Matcher(O.Grammar(ebnf))
    m = B.Matcher(g)
    batch = B.Batch([m])
    mask = torch.zeros((1, tok.words), dtype=torch.int32, device="cuda")
    mask2 = torch.zeros((1, tok.words), dtype=torch.int32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    ids = torch.zeros(1, dtype=torch.int32, device="cuda")
    for piece in list(feed) + [None]:
        batch.fill_next_token_bitmask(mask.data_ptr(), tok.words, st.data_ptr())
        ref = om.mask(ov)
        assert int(st.cpu()[0]) == 0 and np.array_equal(mask.cpu().numpy().view(np.uint32)[0], ref), piece
        if static_too:
            batch.fill_next_token_bitmask_static(mask2.data_ptr(), tok.words, st.data_ptr())
            assert int(st.cpu()[0]) == 0 and np.array_equal(mask2.cpu().numpy().view(np.uint32)[0], ref), piece
        if piece is None:
            break
        ids[0] = toks.index(piece)
        batch.accept_token(ids.data_ptr(), st.data_ptr())
        assert int(st.cpu()[0]) == 0, piece
        assert om.accept_token(ov, toks.index(piece)) == 1
    m.close(); g.close(); tok.close()


def test_item_sets_beyond_the_fast_path():
    """Sixty alternatives that all start with the same byte give Earley sets of sixty items, more than the fixed
    arrays of a token walk hold: the cache is built by the exact slow path, the token is accepted through the
    matcher's large scratch, the step plan that does not fit makes the fill walk the whole vocabulary, and the walks
    that overflow there are redone one by one -- every mask still equals the oracle's, through both fill paths."""
    torch, engine = _engine()
    toks = [bytes([b]) for b in range(256)] + [b"xa", b"xab", b"xq7", b"x", b"xa9!", b"q7", b"b3!", b""]
    toks += [b"\xfe\xff%d" % i for i in range(-len(toks) % 32)]
    eos = toks.index(b"")
    rules = "\n".join('alt%d ::= "x" [a-z]* "%d" "!"?' % (i, i % 10) for i in range(60))
    ebnf = "root ::= " + " | ".join("alt%d" % i for i in range(60)) + "\n" + rules + "\n"
    tok = B.Tokenizer(toks, eos)
    g = B.Grammar(tok, "ebnf", ebnf, inline_max_states=0)
    ov = O.Vocab(toks, eos)
    tb, _ = _oracle_tables(g)
    for s_ in tb.scannable_states()[::7]:
        _check_entry(g, tb, ov, s_, tok.words)
    g.close(); tok.close()
    _drive(ebnf, toks, eos, [b"x", b"a", b"q7", b"!"], static_too=True)
    _drive(ebnf, toks, eos, [b"xab", b"b3!"], static_too=True)


def test_more_entries_to_check_than_the_plan_holds():
    """Forty rules predicted at one position, each with tokens that run past its end: more (state, origin) entries
    with uncertain tokens than the step plan lists.  The fill then takes the mask from the plain definition."""
    toks = [bytes([b]) for b in range(256)] + [b"a0;", b"b1;;", b"c2", b"a0", b";", b"z9;a", b"m3;m", b""]
    toks += [b"\xfe\xff%d" % i for i in range(-len(toks) % 32)]
    eos = toks.index(b"")
    letters = "abcdefghijklmnopqrstuvwxyzABCDEFGHIJKLMN"
    rules = "\n".join('r%d ::= "%s" [0-9]+' % (i, letters[i]) for i in range(40))
    ebnf = 'root ::= (item ";")+\nitem ::= ' + " | ".join("r%d" % i for i in range(40)) + "\n" + rules + "\n"
    _drive(ebnf, toks, eos, [b"a0;", b"c2", b";", b"m3;m", b"7", b";"], static_too=True)


def test_threaded_compile_into_one_pool_builds_the_same_cache():
    """Grammars compiled from eight threads into a shared pool: the same entries as from one thread, and
    between them exactly as many built + reused entries (who builds a shared rule is a matter of timing)."""
    torch, engine = _engine()
    w = inputs.make_workload("C3", batch=12, steps=2, vocab_size=8192)
    a = engine.Session(w, compile_threads=8)
    b = engine.Session(w, compile_threads=1)
    sa, sb = [g.stats() for g in a.grammars], [g.stats() for g in b.grammars]
    total = lambda st: sum(x["n_entries_built"] + x["n_entries_reused"] + x["n_entries_shared"] for x in st)
    assert total(sa) == total(sb)
    assert sum(x["n_entries_built"] for x in sa) == sum(x["n_entries_built"] for x in sb)
    for ga, gb in zip(a.grammars, b.grammars):
        _same_entries(ga, gb, stride=37)
    a.close(); b.close()


def test_next_fill_work_counts_the_plan():
    """The measurement call: merged entries, uncertain candidates and the row of the next fill."""
    torch, engine = _engine()
    w = inputs.make_workload("C5", batch=2, steps=12, vocab_size=8192)
    s = engine.Session(w)
    for step in range(12):
        fw = s.matchers[0].next_fill_work(s.stream())
        assert fw["row_bytes"] == 4 * s.W and fw["n_missing"] == 0
        assert fw["n_merge"] >= 1 and fw["merge_bytes"] > 0
        assert fw["check_bytes"] == 12 * fw["check_tokens"] and fw["n_check"] <= fw["n_merge"] * 2 + 2
        s.fill()
        s.accept([w.trajectories[b][step] for b in range(s.n)])
        for b in range(s.n):
            if w.trajectories[b][step] == w.vocab.eos_id:
                s.reset(b)
    s.close()


def test_tool_pool_requests_share_the_tools_they_have_in_common():
    """Inter-request dynamism (Section 4.1): every request offers its own subset of one tool pool.  The masks are
    exact, and requests compiled later find the entries of the tools that earlier requests already offered."""
    torch, engine = _engine()
    w = inputs.make_workload("P100", batch=6, steps=40, vocab_size=8192)
    names = [set(t["tag"] for t in json.loads(g.text)["tags"]) for g in w.grammars]
    assert all(len(n) == 100 for n in names) and len(set.union(*names)) > 300 and any(names[0] & n for n in names[1:])
    _run_trajectories(w, {0, 13, 39}, check_requests={2})
    s = engine.Session(w, compile_threads=1)
    stats = [g.stats() for g in s.grammars]
    assert stats[0]["n_entries_reused"] < stats[-1]["n_entries_reused"]          # the pool fills up as requests arrive
    assert sum(x["n_entries_reused"] for x in stats[1:]) > 0
    s.close()


def test_changing_batch_compositions_need_no_allocation_and_no_device_synchronisation():
    """Continuous batching: every step one request leaves the batch and another joins, so every step's list of
    matchers is new to the library.  Masks and accepts stay exact, and after the first steps the calls allocate no
    device memory (the per-batch tables are a fixed set of slots that are reused)."""
    torch, engine = _engine()
    w = inputs.make_workload("C3", batch=12, steps=200, vocab_size=8192)
    s = engine.Session(w)
    ov, _, oms = _oracle_side(w)
    n = s.n
    pos = [0] * n                                         # next trajectory step of every request
    mask = torch.zeros((8, s.W), dtype=torch.int32, device=s.device)
    st = torch.zeros(8, dtype=torch.int32, device=s.device)
    ids = torch.zeros(8, dtype=torch.int32, device=s.device)
    free_after_warmup = None
    try:
        for step in range(200):
            members = [(step + k) % n for k in range(8)]          # a window of 8 requests that slides by one every step
            batch = B.Batch([s.matchers[b] for b in members])
            batch.fill_next_token_bitmask(mask.data_ptr(), s.W, st.data_ptr(), s.stream())
            got = mask.cpu().numpy().view(np.uint32)
            assert (st.cpu().numpy() == 0).all()
            toks = []
            for k, b in enumerate(members):
                if step % 5 == 0 or k == 7:
                    assert np.array_equal(got[k], oms[b].mask(ov)), (step, b)
                t = w.trajectories[b][pos[b] % w.steps]
                pos[b] += 1
                toks.append(t)
            ids.copy_(torch.tensor(toks, dtype=torch.int32))
            batch.accept_token(ids.data_ptr(), st.data_ptr(), s.stream(), restart_on_eos=True)
            assert (st.cpu().numpy() == 0).all(), step
            for k, b in enumerate(members):
                if oms[b].accept_token(ov, toks[k]) == 2:
                    oms[b].reset()
            if step == 20:
                torch.cuda.synchronize()
                free_after_warmup = torch.cuda.mem_get_info()[0]
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_after_warmup
    finally:
        s.close()
