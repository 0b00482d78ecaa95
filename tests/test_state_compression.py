"""Repetition state compression (Section 3.6), host side: the classes of automaton states that
share one cache entry, checked against the oracle's own classification of every state.

The library keeps a bounded repetition as explicit states and shares a cache entry between the
states of a rule that agree when unrolled as deep as the longest token.  The oracle knows nothing
about classes: it classifies every (state, token) pair from the exported tables, so equal rows
inside a class is a statement about the equivalence, not about the code that computed it.
"""
import json

import numpy as np
import pytest

from oracle import oracle as O
from oracle import schema_ebnf as SE
from paper_2601_04426_b200 import binding as B
from paper_2601_04426_b200 import inputs
from test_frontend import tables_of


def _bounded_schema(n):
    return json.dumps({"type": "object", "properties": {
        "s": {"type": "string", "minLength": n // 2, "maxLength": n},
        "a": {"type": "array", "items": {"type": "integer"}, "maxItems": n // 4},
        "b": {"type": "array", "items": {"type": "string", "maxLength": 3}, "minItems": 2, "maxItems": n // 4}},
        "required": ["s", "a", "b"]})


def _vocab(size=1536):
    v = inputs.config_vocab("C1", size)
    return v, O.Vocab(v.tokens, v.eos_id, v.special_ids), max(len(t) for t in v.tokens)


@pytest.mark.parametrize("kind,text", [
    ("json_schema", _bounded_schema(48)),
    ("ebnf", 'root ::= "[" item{3,40} "]" tail{0,30}\nitem ::= [a-c] | "(" item{1,2} ")"\ntail ::= "ab" | "a"'),
    ("ebnf", 'root ::= ("x" | "yz"){20,60} "!" [0-9]{0,25}'),
])
def test_states_of_one_class_have_identical_cache_rows(kind, text):
    v, ov, max_len = _vocab()
    tb, g = tables_of(kind, text)
    rep = g.state_classes(max_len)
    scannable = tb.scannable_states()
    rows = {}
    shared = 0
    for s in scannable:
        r = int(rep[s])
        assert r <= s and rep[r] == r
        assert tb.a["state_rule"][r] == tb.a["state_rule"][s]
        if r not in rows:
            rows[r] = tb.classify(ov, r)
        if r != s:
            shared += 1
            assert np.array_equal(tb.classify(ov, s), rows[r]), (s, r)
    assert shared > 0 and len(rows) < len(scannable)


def test_class_count_does_not_grow_with_the_bound():
    """Past a few token lengths, a larger bound adds states but no classes: the entries to build
    stay bounded (the point of Section 3.6)."""
    counts = {}
    for n in (128, 256, 1024):
        g = B.Grammar(None, "json_schema", _bounded_schema(n))
        rep = g.state_classes(12)
        counts[n] = (len(np.unique(rep)), len(rep))
    assert counts[128][0] == counts[256][0] == counts[1024][0]
    assert counts[1024][1] > 6 * counts[128][1]
    assert counts[1024][0] < counts[1024][1] // 20


def test_too_shallow_a_depth_would_merge_states_that_tokens_tell_apart():
    """The depth matters: with classes one edge deep, states near the end of a repetition share a
    class with states in its middle although a two-byte token separates them."""
    v, ov, max_len = _vocab()
    tb, g = tables_of("ebnf", 'root ::= [a-z]{0,30} "!"')
    shallow, deep = g.state_classes(1), g.state_classes(max_len)
    mixed = 0
    for s in tb.scannable_states():
        r = int(shallow[s])
        if r != s and not np.array_equal(tb.classify(ov, s), tb.classify(ov, r)):
            mixed += 1
            assert deep[s] != deep[r]
    assert mixed > 0


def test_masks_from_shared_rows_equal_the_plain_definition():
    """Merge rule over per-class rows: along a trajectory that runs through long repetitions, the
    mask assembled from the representatives' rows and a full check of the uncertain tokens equals
    the oracle's plain mask."""
    w = inputs.make_workload("R256", batch=2, steps=150, vocab_size=1536)
    ov = O.Vocab(w.vocab.tokens, w.vocab.eos_id, w.vocab.special_ids)
    max_len = max(len(t) for t in w.vocab.tokens)
    for b in range(2):
        spec = w.grammars[w.request_grammar[b]]
        tb, g = tables_of(spec.kind, spec.text)
        rep = g.state_classes(max_len)
        scannable = set(tb.scannable_states())
        om = O.Matcher(O.Grammar(SE.grammar_text(spec.kind, spec.text)))
        tm = O.TableMatcher(tb)
        rows = {}
        for step, tok in enumerate(w.trajectories[b]):
            if step % 7 == 0:
                ref = O.unpack_bits(om.mask(ov), ov.size)
                acc = np.zeros(ov.size, bool)
                unc = np.zeros(ov.size, bool)
                for s in sorted({s for s, _ in tm.get_set(tm.num_sets() - 1)} & scannable):
                    r = int(rep[s])
                    if r not in rows:
                        rows[r] = tb.classify(ov, r)
                    acc |= rows[r] == 1
                    unc |= rows[r] == 2
                # accepted rows are allowed outright; what is allowed beyond them is uncertain somewhere
                assert ref[acc].all(), step
                assert not (ref & ~acc & ~unc).any(), step
            if tok == w.vocab.eos_id:
                assert om.accept_token(ov, tok) == 2
                om.reset(); tm.reset()
            else:
                assert om.accept_token(ov, tok) == 1
                assert tm.accept_bytes(w.vocab.tokens[tok])


# ---- GPU: the library's shared entries and the masks built from them -----------------------

def _entry_key(e):
    return (e["kind"], e["n_accepted"], e["n_uncertain"], e["list"].tobytes(), e["uncertain"].tobytes(),
            e["bitset"].tobytes() if e["kind"] == B.XG_STORE_BITSET else b"")


@pytest.mark.gpu
def test_gpu_shared_entries_match_oracle_rows_and_the_uncompressed_build():
    """Every scannable state's entry -- its own or its class's -- equals the oracle's row for that
    very state, and equals what a compile with compression switched off builds for it."""
    w = inputs.make_workload("R256", batch=1, steps=2, vocab_size=4096)
    v = w.vocab
    ov = O.Vocab(v.tokens, v.eos_id, v.special_ids)
    tok = B.Tokenizer(v.tokens, v.eos_id, v.special_ids)
    spec = w.grammars[0]
    # (repeat_threshold=-1: the repetitions expanded into explicit states, which is what this sharing is about)
    g = B.Grammar(tok, spec.kind, spec.text, repeat_threshold=-1)
    plain = B.Grammar(tok, spec.kind, spec.text, state_compression=False, repeat_threshold=-1)
    tb, _ = tables_of(spec.kind, spec.text)
    rep = g.state_classes()
    st, st_plain = g.stats(), plain.stats()
    scannable = tb.scannable_states()
    assert st["n_entries_built"] + st["n_entries_shared"] == len(scannable) == st_plain["n_entries_built"]
    assert st_plain["n_entries_shared"] == 0 and st["n_entries_built"] * 4 < len(scannable)
    assert st["cache_bytes"] * 4 < st_plain["cache_bytes"]
    members = [s for s in scannable if rep[s] != s]
    for s in members[::23] + [s for s in scannable if rep[s] == s][::5]:
        e = g.cache_entry(s)
        cls = tb.classify(ov, s)
        assert set(e["uncertain"].tolist()) == set(np.nonzero(cls == 2)[0].tolist()), s
        assert e["n_accepted"] == int((cls == 1).sum()), s
        assert _entry_key(e) == _entry_key(plain.cache_entry(s)), s
    g.close(); plain.close(); tok.close()


@pytest.mark.gpu
@pytest.mark.parametrize("name,vsize,steps", [("R256", 16384, 200), ("R1024", 8192, 120)])
def test_gpu_masks_through_long_repetitions_bit_exact(name, vsize, steps):
    """With the repetitions expanded into explicit states whose cache entries are shared."""
    from test_gpu_parity import _run_trajectories
    w = inputs.make_workload(name, batch=8, steps=steps, vocab_size=vsize)
    compared = _run_trajectories(w, set(range(0, steps, 9)), check_requests={1, 2}, repeat_threshold=-1)
    assert compared > steps
