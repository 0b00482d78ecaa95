"""Host logic of the library (no GPU): the grammar front end's tables, checked against the oracle.

The oracle reads the grammar text with its own parser and runs a textbook Earley recogniser; the
library lowers the same text to per-rule automata.  The oracle's table interpreter runs those
tables, so language and mask equality here means the two front ends agree.
"""
import ctypes
import json
import os

import numpy as np
import pytest

from oracle import oracle as O
from oracle import schema_ebnf as SE
from paper_2601_04426_b200 import binding as B
from paper_2601_04426_b200 import inputs
from test_oracle_earley import CFG_CASES, REGEX_CASES, all_strings


def tables_of(kind, text, **kw):
    g = B.Grammar(None, kind, text, **kw)
    t = g.tables()
    scal = {k: t.pop(k) for k in ("n_rules", "n_states", "n_classes", "root_rule", "root_nullable")}
    return O.Tables(scal["n_rules"], scal["n_states"], scal["n_classes"], scal["root_rule"], scal["root_nullable"], **t), g


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(B.lib_path()) if os.path.exists(B.lib_path()) else B.lib()
    header = open(os.path.join(os.path.dirname(B.lib_path()), "..", "include", "xg.h")).read()
    import re
    declared = set(re.findall(r"\b(xg_[a-z_]+)\s*\(", header)) - {"xg_status_t"}
    assert declared == set(B.EXPORTS), declared ^ set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def _same_language(ebnf, alphabet, max_len, **kw):
    og = O.Grammar(ebnf)
    tb, _ = tables_of("ebnf", ebnf, **kw)
    for s in all_strings(alphabet, max_len):
        data = s.encode()
        tm = O.TableMatcher(tb)
        ok = tm.accept_bytes(data)
        assert ok == O.is_prefix(og, data), (ebnf, s)
        if ok:
            assert tm.can_terminate() == O.accepts(og, data), (ebnf, s)


@pytest.mark.parametrize("inline", [0, 12])
def test_tables_same_language_as_oracle_on_small_grammars(inline):
    for name, ebnf, _, alphabet, _ in CFG_CASES:
        _same_language(ebnf, alphabet, 6, inline_max_states=inline)
    for ebnf, _, alphabet in REGEX_CASES:
        _same_language(ebnf, alphabet, 6, inline_max_states=inline)
    _same_language('root ::= TagDispatch(("ab", g), stop_strs=("xb")) "!"\ng ::= "a"', "abx!", 6, inline_max_states=inline)
    _same_language('root ::= TagDispatch(("ab", g))\ng ::= "x" "x"?', "abx", 7, inline_max_states=inline)
    _same_language('root ::= "q"? TagDispatch(("<a>", r0), ("<<b", r1)) \nr0 ::= "0"\nr1 ::= "1" root?', "<>ab01q", 5, inline_max_states=inline)
    # a text channel: a TagDispatch without tags that runs to its stop string, nested in a dispatching one
    _same_language('root ::= TagDispatch(("<a", body), stop_strs=("!"))\nbody ::= TagDispatch(stop_strs=("a>", ">>"))', "<a>!", 7, inline_max_states=inline)


def test_tables_invariants():
    for name in ("C1", "C3", "C4", "C5"):
        w = inputs.make_workload(name, batch=1, steps=2)
        g = B.Grammar(None, w.grammars[0].kind, w.grammars[0].text)
        t = g.tables()
        S, R = t["n_states"], t["n_rules"]
        assert len(t["state_rule"]) == S and len(t["rule_start"]) == R
        assert all(t["state_rule"][t["rule_start"][r]] == r for r in range(R))
        # no rule accepts the empty string; every rule has an accepting state
        assert not any(t["state_final"][t["rule_start"][r]] for r in range(R))
        for r in range(R):
            assert t["state_final"][t["state_rule"] == r].any()
        # deterministic: byte classes leaving one state are pairwise disjoint, references distinct
        bits = t["class_bits"].reshape(-1, 8)
        for s in range(S):
            acc = np.zeros(8, dtype=np.uint32)
            for e in range(t["cedge_begin"][s], t["cedge_begin"][s + 1]):
                c = bits[t["cedge_class"][e]]
                assert c.any() and not (acc & c).any()
                acc |= c
            refs = t["redge_rule"][t["redge_begin"][s]:t["redge_begin"][s + 1]]
            assert len(set(refs.tolist())) == len(refs)
        assert (t["cedge_target"] < S).all() and (t["redge_target"] < S).all() and (t["redge_rule"] < R).all()


def _mutate(rng, doc, alphabet):
    pos = rng.below(len(doc))
    b = bytes([alphabet[rng.below(len(alphabet))]])
    kind = rng.below(3)
    return doc[:pos] + b + doc[pos + 1:] if kind == 0 else (doc[:pos] + doc[pos + 1:] if kind == 1 else doc[:pos] + b + doc[pos:])


@pytest.mark.parametrize("name", ["C1", "C2", "C3", "C4", "C5", "T20", "H16", "R256", "P10"])
def test_workload_grammars_same_language_as_oracle(name):
    w = inputs.make_workload(name, batch=3, steps=40)
    rng = inputs.Rng(17)
    alphabet = b'{}[]:,"\\ -.0123456789etrufalsn<>/_\xc3\xa9'
    for gi in sorted(set(w.request_grammar)):
        spec = w.grammars[gi]
        og = O.Grammar(SE.grammar_text(spec.kind, spec.text))
        tb, _ = tables_of(spec.kind, spec.text)
        for b in [i for i, x in enumerate(w.request_grammar) if x == gi]:
            for doc in w.documents[b][:2]:
                tm = O.TableMatcher(tb)
                assert tm.accept_bytes(doc), doc
                assert tm.can_terminate() == O.accepts(og, doc)
                for _ in range(25):
                    mut = _mutate(rng, doc, alphabet)
                    tm = O.TableMatcher(tb)
                    ok = tm.accept_bytes(mut)
                    assert ok == O.is_prefix(og, mut), mut
                    if ok:
                        assert tm.can_terminate() == O.accepts(og, mut), mut


@pytest.mark.parametrize("name,vsize,steps", [("C1", 2048, 40), ("C4", 2048, 60), ("C5", 4096, 30), ("T5", 2048, 50), ("H16", 2048, 70)])
def test_masks_plain_equals_merged_equals_oracle(name, vsize, steps):
    """The cache classification plus the merge rule reproduces the plain definition, step by step."""
    w = inputs.make_workload(name, batch=1, steps=steps, vocab_size=vsize)
    spec = w.grammars[0]
    ov = O.Vocab(w.vocab.tokens, w.vocab.eos_id, w.vocab.special_ids)
    og = O.Grammar(SE.grammar_text(spec.kind, spec.text))
    tb, _ = tables_of(spec.kind, spec.text)
    om, tm = O.Matcher(og), O.TableMatcher(tb)
    checked_total = 0
    for step, tok in enumerate(w.trajectories[0]):
        ref = om.mask(ov)
        assert np.array_equal(tm.mask_plain(ov), ref), step
        merged, n_checked = tm.mask_merged(ov)
        assert np.array_equal(merged, ref), step
        checked_total += n_checked
        if tok == w.vocab.eos_id:
            assert om.accept_token(ov, tok) == 2
            om.reset(); tm.reset()
        else:
            assert om.accept_token(ov, tok) == 1
            assert tm.accept_bytes(w.vocab.tokens[tok])
    assert checked_total < steps * vsize          # the cache decides most tokens


def test_classification_partition_and_soundness():
    """Accepted / uncertain / rejected partition the vocabulary; accepted tokens are allowed in
    every state that contains the position, rejected ones are allowed only through other items."""
    w = inputs.make_workload("C5", batch=1, steps=25, vocab_size=2048)
    ov = O.Vocab(w.vocab.tokens, w.vocab.eos_id, w.vocab.special_ids)
    tb, _ = tables_of("ebnf", w.grammars[0].text)
    tm = O.TableMatcher(tb)
    cls_cache = {}
    for tok in w.trajectories[0]:
        if tok == w.vocab.eos_id:
            tm.reset()
            continue
        bits = O.unpack_bits(tm.mask_plain(ov), ov.size)
        states = sorted({s for s, _ in tm.get_set(tm.num_sets() - 1) if s in set(tb.scannable_states())})
        union_acc = np.zeros(ov.size, bool)
        union_unc = np.zeros(ov.size, bool)
        for s in states:
            if s not in cls_cache:
                cls_cache[s] = tb.classify(ov, s)
            c = cls_cache[s]
            assert set(np.unique(c)) <= {0, 1, 2}
            assert not bits[(c == 1) & ~bits].any() and bits[c == 1].all()
            union_acc |= c == 1
            union_unc |= c == 2
        assert not (bits & ~union_acc & ~union_unc)[:ov.size].any()      # allowed => accepted or uncertain somewhere
        tm.accept_bytes(w.vocab.tokens[tok])


def test_classification_against_hand_worked_table():
    """Section 3.4 on paper: every token at every scannable state of a two-rule grammar, from both
    sides -- a token wrongly called uncertain (an inner rule ended, the state's own did not) fails
    here just as one wrongly called accepted or rejected."""
    from golden_util import load_classify_fixture, state_at_path
    ebnf, tokens, cases = load_classify_fixture("classify_bracket_item.txt")
    ov = O.Vocab([t.encode() for t in tokens], tokens.index(""))
    tb, g = tables_of("ebnf", ebnf, inline_max_states=0)
    t = g.tables()
    assert t["n_rules"] == 2                              # `item` was kept as a rule of its own
    states = [state_at_path(t, path) for path, _, _ in cases]
    assert sorted(states) == tb.scannable_states()        # the fixture covers every scannable state
    for s, (path, acc, unc) in zip(states, cases):
        cls = tb.classify(ov, s)
        assert sorted(tokens[i] for i in np.nonzero(cls == 1)[0]) == sorted(acc), path
        assert sorted(tokens[i] for i in np.nonzero(cls == 2)[0]) == sorted(unc), path


def test_front_end_errors():
    cases = [("ebnf", 'root ::= "a', B.XG_ERR_PARSE), ("ebnf", "root ::= missing", B.XG_ERR_PARSE), ("ebnf", 'x ::= "a"', B.XG_ERR_PARSE),
             ("ebnf", 'root ::= "a"{3,2}', B.XG_ERR_PARSE), ("json_schema", "{", B.XG_ERR_PARSE),
             ("json_schema", json.dumps({"type": "string", "pattern": "a"}), B.XG_ERR_UNSUPPORTED),
             ("json_schema", json.dumps({"type": "object", "properties": {"a": {"type": "null"}}, "required": []}), B.XG_ERR_UNSUPPORTED),
             ("tag_dispatch", json.dumps({"tags": []}), B.XG_ERR_PARSE)]
    for kind, text, status in cases:
        with pytest.raises(B.XgError) as e:
            B.Grammar(None, kind, text)
        assert e.value.status == status, (text, e.value)
        assert str(e.value)


def test_front_end_limits():
    with pytest.raises(B.XgError) as e:
        B.Grammar(None, "ebnf", "root ::= " + "(" * 300 + '"a"' + ")" * 300)
    assert e.value.status == B.XG_ERR_PARSE
    with pytest.raises(B.XgError) as e:
        B.Grammar(None, "ebnf", 'root ::= ("abcdefgh"{1000}){1000}')
    assert e.value.status == B.XG_ERR_CAPACITY
    g = B.Grammar(None, "ebnf", 'root ::= [a-z]{0,300} "!"')          # a long bounded repetition is fine
    assert g.stats()["n_states"] >= 300


def test_just_in_time_and_class_calls_on_the_host():
    """What needs no device: the service call over nothing or over grammars without a cache is a no-op, the
    class export checks its arguments, and the just-in-time options do not change the front end's tables."""
    assert B.jit_service([], 0, False) == {"n_built": 0, "n_pool_hits": 0, "n_in_flight": 0, "n_missing": 0}
    text = 'root ::= "[" [a-z]{2,40} "]"'
    plain = B.Grammar(None, "ebnf", text)
    jit = B.Grammar(None, "ebnf", text, jit=True, jit_precompute=3, state_compression=False)
    assert B.jit_service([plain, jit], 0, True)["n_missing"] == 0        # compiled without a tokenizer: not just-in-time grammars
    ta, tb = plain.tables(), jit.tables()
    assert all(np.array_equal(ta[k], tb[k]) for k in ta)
    with pytest.raises(B.XgError) as e:
        plain.state_classes(-1)                                          # the default depth needs a tokenizer
    assert e.value.status == B.XG_ERR_INVALID_ARG
    rep0, rep9 = plain.state_classes(0), plain.state_classes(9)
    assert len(np.unique(rep0)) <= len(np.unique(rep9)) <= len(rep9)
    assert (rep9 <= np.arange(len(rep9))).all() and (rep9[rep9] == rep9).all()


def test_device_entry_points_fail_loudly_without_a_gpu():
    """No CPU fallback: without a CUDA device the device entry points return XG_ERR_CUDA."""
    try:
        import torch
        if torch.cuda.is_available():
            pytest.skip("a GPU is present")
    except ImportError:
        pass
    with pytest.raises(B.XgError) as e:
        B.Tokenizer([b"a", b"b", b""], eos_id=2)
    assert e.value.status == B.XG_ERR_CUDA and "vocabulary upload" in str(e.value)


def test_schema_lowerings_agree():
    """The library's schema -> grammar text and the oracle's, each read by the oracle's parser,
    accept the same documents (the texts themselves differ)."""
    rng = inputs.Rng(3)
    for _ in range(6):
        schema = inputs.make_object_schema(rng, rng.randint(2, 6), 2)
        text = json.dumps(schema)
        ga = O.Grammar(SE.schema_to_ebnf(text))
        tb, _ = tables_of("json_schema", text)
        for _ in range(5):
            doc = inputs.sample_document(schema, rng, wide=True).encode()
            assert O.accepts(ga, doc)
            tm = O.TableMatcher(tb)
            assert tm.accept_bytes(doc) and tm.can_terminate()


# ---------------------------------------------------------------------------------------
# structural hash (Section 3.3, Algorithms 1 and 2)
# ---------------------------------------------------------------------------------------

def _hashes(ebnf, root="root"):
    g = B.Grammar(None, "ebnf", ebnf, root=root, inline_max_states=0)
    return g.rule_hashes()


def test_structural_hash_ignores_names_and_order():
    a = _hashes('root ::= "x" item "y" | "z"\nitem ::= [0-9]+ "." [a-f]')
    b = _hashes('digits ::= [0-9]+ "." [a-f]\nroot ::= "z" | "x" digits "y"')
    assert a[0] == b[0] and a[1] == b[1]
    # the same sub-rule inside a different grammar keeps its hash (cross-grammar reuse)
    c = _hashes('root ::= "{" item "}" item\nitem ::= [0-9]+ "." [a-f]')
    assert c[1] == a[1] and c[0] != a[0]


def test_structural_hash_sees_single_edits():
    base = 'root ::= "x" item "y"\nitem ::= [0-9]+ "." [a-f]'
    h0 = _hashes(base)
    for edit in ['root ::= "x" item "z"\nitem ::= [0-9]+ "." [a-f]',
                 'root ::= "x" item "y"\nitem ::= [0-8]+ "." [a-f]',
                 'root ::= "x" item "y"\nitem ::= [0-9]+ "." [a-f]?',
                 'root ::= "x" item "y"\nitem ::= [0-9]* "." [a-f]']:
        h = _hashes(edit)
        assert h[0] != h0[0]
    # an edit inside the referenced rule changes both hashes; an edit in the user only the user's
    h = _hashes('root ::= "x" item "q"\nitem ::= [0-9]+ "." [a-f]')
    assert h[1] == h0[1] and h[0] != h0[0]


def test_structural_hash_on_cycles():
    """Members of a reference cycle get distinct hashes, stable under renaming and under which
    member is the root (Algorithm 2: the fold starts at the member being hashed)."""
    ring = 'a ::= "1" b | "x"\nb ::= "2" c | "y"\nc ::= "3" a | "z"'
    ha = _hashes(ring, root="a")
    assert len(set(ha.tolist())) == 3
    hb = _hashes(ring, root="b")
    assert set(ha.tolist()) == set(hb.tolist())
    renamed = 'p ::= "1" q | "x"\nq ::= "2" r | "y"\nr ::= "3" p | "z"'
    assert set(_hashes(renamed, root="p").tolist()) == set(ha.tolist())
    other = 'a ::= "1" b | "x"\nb ::= "2" c | "y"\nc ::= "4" a | "z"'
    assert not set(_hashes(other, root="a").tolist()) & set(ha.tolist())
    # One state with two references into its own cycle: their order in the canonical form must come from the
    # referenced rules' structure, not from their indices in this grammar -- declared in another order (and with an
    # unrelated rule in front, which shifts every index) the cycle hashes the same.
    # (inline_max_states=0 keeps every rule: folding rules of a cycle into each other would hide the references)
    knot = 'top ::= "<" (left | right) ">"\nleft ::= "l" top "1" | "e"\nright ::= "r" top "22" | "f" "g"'
    tonk = 'pad ::= "p"\ntop ::= "<" (right | left) ">" \nright ::= "f" "g" | "r" top "22"\nleft ::= "e" | "l" top "1"\nmain ::= pad top'
    h1 = B.Grammar(None, "ebnf", knot, root="top", inline_max_states=0).rule_hashes()
    h2 = B.Grammar(None, "ebnf", tonk, root="main", inline_max_states=0).rule_hashes()
    assert len(h1) == 3 and set(h1.tolist()) <= set(h2.tolist())


def test_front_end_is_reentrant():
    """Several threads compiling at once get the tables a single thread gets."""
    from concurrent.futures import ThreadPoolExecutor
    w = inputs.make_workload("C3", batch=12, steps=2)

    def tables(spec):
        t = B.Grammar(None, spec.kind, spec.text).tables()
        return {k: (v.copy() if hasattr(v, "copy") else v) for k, v in t.items()}

    serial = [tables(g) for g in w.grammars]
    with ThreadPoolExecutor(max_workers=6) as ex:
        threaded = list(ex.map(tables, w.grammars * 3))
    for i, t in enumerate(threaded):
        ref = serial[i % len(serial)]
        assert all(np.array_equal(ref[k], t[k]) for k in ref), i
