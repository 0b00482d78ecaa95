"""Counted repetitions (Section 3.6: the parser state (R{l,r}, k)) -- CPU tests.

The front end keeps X{l,r} with a large r as one copy of X whose items carry the count k.  The oracle's table
interpreter runs such tables with the count in the item; here it is pinned against the oracle's grammar-text
recogniser, which knows nothing about counts (it expands every repetition), by brute force over all short strings
and along sampled documents, and the library's tables are checked for what the section promises: a number of states
that does not grow with the bound.
"""
import numpy as np
import pytest

from oracle import oracle as O
from oracle import schema_ebnf as SE
from paper_2601_04426_b200 import binding as B
from paper_2601_04426_b200 import inputs
from test_frontend import tables_of
from test_oracle_earley import all_strings

# (grammar text, alphabet, longest string tried)
COUNTED_CASES = [
    ('root ::= "a"{2,5}', "ab", 7),                                   # unary: the pin the section's algorithm is checked on
    ('root ::= "a"{0,4}', "a", 6),                                    # lower bound 0: the rule may be skipped
    ('root ::= "<" "a"{3,6} "a" ">"', "a<>", 9),                      # the same byte continues after the repetition
    ('root ::= "[" ("ab" | "c"){1,4} "]"', "abc[]", 8),               # bodies of different lengths
    ('root ::= ([a-b]+ ","){2,3} "."', "ab,.", 8),                    # a body that loops in itself
    ('root ::= ("a"? "b"?){2,4} "!"', "ab!", 7),                      # a body that may be empty
    ('root ::= (item ","){1,3} item\nitem ::= "x" | "(" root ")"', "x,()", 8),      # recursion through the body
    ('root ::= ("a" "b"{2,3}){2,3}', "ab", 9),                        # a counted repetition inside another
    ('root ::= "a"{3,3} | "a"{5,5} "b"', "ab", 7),                    # two of them side by side from one state
    ('root ::= ("a" | "aa"){2,3} "a"', "a", 8),                       # ambiguous: several counts alive at once
    ('root ::= TagDispatch(("<a", g), stop_strs=("!"))\ng ::= "x"{2,4} ">"', "<ax>!", 6),      # inside a dispatched grammar
]


def _counted(text, depth, threshold=2, **kw):
    return tables_of("ebnf", text, repeat_threshold=threshold, repeat_depth=depth, **kw)


@pytest.mark.parametrize("depth", [1, 3])
def test_counted_tables_same_language_as_plain_expansion(depth):
    """Brute force: the counted tables accept exactly the viable prefixes and sentences of the expanded grammar."""
    for text, alphabet, max_len in COUNTED_CASES:
        og = O.Grammar(text)
        tb, g = _counted(text, depth)
        assert tb.counted, text                                        # the construct was really kept as a counter
        for s in all_strings(alphabet, max_len):
            data = s.encode()
            tm = O.TableMatcher(tb)
            ok = tm.accept_bytes(data)
            assert ok == O.is_prefix(og, data), (text, s)
            if ok:
                assert tm.can_terminate() == O.accepts(og, data), (text, s)


def test_counted_tables_equal_expanded_tables_as_languages():
    """The same front end with counting switched off gives tables of the same language (the count is the only change)."""
    for text, alphabet, max_len in COUNTED_CASES[:6]:
        tb, _ = _counted(text, 2)
        tp, _ = tables_of("ebnf", text, repeat_threshold=-1)
        assert not tp.counted
        for s in all_strings(alphabet, max_len - 1):
            a, b = O.TableMatcher(tb), O.TableMatcher(tp)
            ok = a.accept_bytes(s.encode())
            assert ok == b.accept_bytes(s.encode()), (text, s)
            if ok:
                assert a.can_terminate() == b.can_terminate(), (text, s)


def test_state_count_does_not_grow_with_the_bound():
    sizes = []
    for bound in (64, 1024, 65536):
        g = B.Grammar(None, "ebnf", 'root ::= "\\"" [a-z0-9 ]{0,%d} "\\""' % bound, build_cache=False, repeat_threshold=64, repeat_depth=16)
        t = g.tables()
        sizes.append((t["n_states"], t["n_records"]))
        assert t["rule_rep_hi"].max() == bound
    assert sizes[0] == sizes[1] == sizes[2], sizes
    expanded = B.Grammar(None, "ebnf", 'root ::= "\\"" [a-z0-9 ]{0,1024} "\\""', build_cache=False, repeat_threshold=-1).tables()
    assert expanded["n_states"] > 1024 > sizes[0][0]


def test_largest_bounds():
    """Bounds up to the grammar text's largest number (10^6) are counted with the same handful of states; beyond that
    the text is refused.  (The count shares the item's 32-bit state word with the state number; a bound that would not
    fit beside a very large grammar's state numbers is XG_ERR_CAPACITY, never a wrong parse.)"""
    ok = B.Grammar(None, "ebnf", 'root ::= "a"{0,1000000}', build_cache=False, repeat_threshold=64, repeat_depth=8)
    assert ok.tables()["rule_rep_hi"].max() == 1000000 and ok.tables()["n_states"] < 10
    with pytest.raises(B.XgError) as e:
        B.Grammar(None, "ebnf", 'root ::= "a"{0,2000000000}', build_cache=False, repeat_threshold=64, repeat_depth=8)
    assert e.value.status == B.XG_ERR_PARSE
    # without the longest token's length nothing is counted
    plain = B.Grammar(None, "ebnf", 'root ::= "a"{0,100}', build_cache=False, repeat_threshold=64)
    assert plain.tables()["rule_rep_hi"].size == 0 and plain.tables()["n_states"] > 100


def test_items_carry_the_count():
    tb, _ = _counted('root ::= "a"{2,9} "b"', 2)
    tm = O.TableMatcher(tb)
    for n in range(1, 8):
        assert tm.accept_bytes(b"a")
        last = tm.num_sets() - 1
        rules = tb.a["state_rule"]
        counts = [k for (s, _), k in zip(tm.get_set(last), tm.get_set_counts(last)) if tb.a["rule_rep_hi"][rules[s]]]
        assert counts and set(counts) == {n - 1}, (n, counts)      # n iterations begun: n - 1 finished before the current one


@pytest.mark.parametrize("name,vsize,steps", [("R256", 2048, 90), ("R1024", 1024, 60)])
def test_masks_with_counted_repetitions_equal_the_plain_definition(name, vsize, steps):
    """On the long-repetition workloads: the counted tables' plain mask, and the mask merged from per-(state, count)
    classifications, both equal the mask of the grammar-text oracle at every step."""
    w = inputs.make_workload(name, batch=1, steps=steps, vocab_size=vsize)
    spec = w.grammars[0]
    ov = O.Vocab(w.vocab.tokens, w.vocab.eos_id, w.vocab.special_ids)
    og = O.Grammar(SE.grammar_text(spec.kind, spec.text))
    depth = max(len(t) for t in w.vocab.tokens)
    tb, g = tables_of(spec.kind, spec.text, repeat_threshold=64, repeat_depth=depth)
    assert tb.counted
    assert g.tables()["n_states"] < 1200
    om, tm = O.Matcher(og), O.TableMatcher(tb)
    for step, tok in enumerate(w.trajectories[0]):
        ref = om.mask(ov)
        assert np.array_equal(tm.mask_plain(ov), ref), step
        if step % 6 == 0:
            merged, _ = tm.mask_merged(ov)
            assert np.array_equal(merged, ref), step
        if tok == w.vocab.eos_id:
            assert om.accept_token(ov, tok) == 2
            om.reset(); tm.reset()
        else:
            assert om.accept_token(ov, tok) == 1
            assert tm.accept_bytes(w.vocab.tokens[tok])


def test_classification_is_the_same_for_every_count_of_a_record():
    """Counts that fall into one record (equally far, up to the longest token, from both bounds) classify every token
    alike; counts in different records near a bound differ somewhere."""
    w = inputs.make_workload("R256", batch=1, steps=2, vocab_size=1024)
    ov = O.Vocab(w.vocab.tokens, w.vocab.eos_id, w.vocab.special_ids)
    depth = max(len(t) for t in w.vocab.tokens)
    text = 'root ::= "\\"" [a-z0-9 ]{40,200} "\\""'
    tb, g = tables_of("ebnf", text, repeat_threshold=64, repeat_depth=depth)
    t = g.tables()
    rep_states = [s for s in tb.scannable_states() if t["rule_rep_hi"][t["state_rule"][s]]]
    assert rep_states
    s = rep_states[0]
    by_record = {}
    for k in list(range(0, 200, 7)) + list(range(20, 42)) + list(range(180, 200)):
        by_record.setdefault(g.record_of(s, k), []).append(k)
    assert len(by_record) > 4 and any(len(v) > 3 for v in by_record.values())
    rows = {}
    for rec, ks in by_record.items():
        cls = [tb.classify(ov, s, count=k, threads=1) for k in ks[:4]]
        for c in cls[1:]:
            assert np.array_equal(c, cls[0]), (rec, ks)
        rows[rec] = cls[0]
    assert not np.array_equal(rows[g.record_of(s, 199)], rows[g.record_of(s, 100)])      # at the upper bound nothing may follow
    assert not np.array_equal(rows[g.record_of(s, 30)], rows[g.record_of(s, 100)])       # below the lower bound the quote may not close


# ---- GPU ------------------------------------------------------------------------------------------------------------

@pytest.mark.gpu
@pytest.mark.parametrize("name,vsize,steps", [("R256", 16384, 200), ("R1024", 8192, 160), ("R4096", 8192, 160)])
def test_gpu_masks_with_counted_repetitions_bit_exact(name, vsize, steps):
    """The default compile counts these workloads' repetitions; every compared mask equals the grammar-text oracle's."""
    from test_gpu_parity import _run_trajectories
    w = inputs.make_workload(name, batch=8, steps=steps, vocab_size=vsize)
    compared = _run_trajectories(w, set(range(0, steps, 9)), check_requests={1, 2})
    assert compared > steps


@pytest.mark.gpu
def test_gpu_counted_repetitions_fused_steps_and_restart():
    from test_gpu_parity import _run_trajectories
    w = inputs.make_workload("R256", batch=4, steps=150, vocab_size=8192)
    assert _run_trajectories(w, set(range(0, 150, 7)), fused=True) > 40
    assert _run_trajectories(w, set(range(0, 150, 11)), restart=True) > 20


@pytest.mark.gpu
def test_gpu_counted_grammar_is_small_and_fast_to_compile():
    """States and records do not depend on the bound (the section's claim); the expanded compile of the same grammar
    has hundreds of times more states."""
    w = inputs.make_workload("R4096", batch=1, steps=2, vocab_size=8192)
    v = w.vocab
    tok = B.Tokenizer(v.tokens, v.eos_id, v.special_ids)
    spec = w.grammars[0]
    counted = B.Grammar(tok, spec.kind, spec.text)
    w2 = inputs.make_workload("R1024", batch=1, steps=2, vocab_size=8192)      # (every bound of it is counted too)
    small = B.Grammar(tok, w2.grammars[0].kind, w2.grammars[0].text)
    expanded = B.Grammar(tok, spec.kind, spec.text, repeat_threshold=-1)
    a, b, c = counted.stats(), small.stats(), expanded.stats()
    # (the two schemas differ in a few literal bytes, nothing else: four times the bounds, about the same states)
    assert abs(a["n_states"] - b["n_states"]) < 20 and a["n_states"] * 100 < c["n_states"]
    assert abs(counted.tables()["n_records"] - small.tables()["n_records"]) < 20
    assert a["frontend_ms"] * 10 < c["frontend_ms"]
    counted.close(); small.close(); expanded.close(); tok.close()


@pytest.mark.gpu
def test_gpu_cache_entries_of_counted_records_match_the_oracle():
    """Per (state, count): the entry of its record equals the oracle's classification from that very count --
    in the middle of the repetition, near both bounds, and at them."""
    from test_gpu_parity import _entry_classes
    w = inputs.make_workload("R256", batch=1, steps=2, vocab_size=8192)
    v = w.vocab
    ov = O.Vocab(v.tokens, v.eos_id, v.special_ids)
    tok = B.Tokenizer(v.tokens, v.eos_id, v.special_ids)
    text = 'root ::= "[" ("\\"" [a-z0-9 ]{40,300} "\\"" ", "){2,80} "]"'
    g = B.Grammar(tok, "ebnf", text)
    t = g.tables()
    scal = {k: t.pop(k) for k in ("n_rules", "n_states", "n_classes", "root_rule", "root_nullable")}
    tb = O.Tables(scal["n_rules"], scal["n_states"], scal["n_classes"], scal["root_rule"], scal["root_nullable"], **t)
    assert tb.counted and (t["rule_rep_hi"] > 0).sum() == 2
    checked = 0
    for s in tb.scannable_states():
        hi = int(t["rule_rep_hi"][t["state_rule"][s]])
        lo = int(t["rule_rep_lo"][t["state_rule"][s]])
        counts = [0] if hi == 0 else sorted({0, 1, lo - 2, lo - 1, lo, (lo + hi) // 2, hi - 13, hi - 2, hi - 1} & set(range(hi)))
        for k in counts:
            ref = tb.classify(ov, s, count=k)
            try:
                cls = _entry_classes(g.cache_entry(g.record_of(s, k)), v.size)
            except B.XgError:
                # a state whose only byte edges start the next iteration has none at the last count: no entry, and
                # the oracle rejects every token there
                assert k == hi - 1 and not ref.any(), (s, k)
                continue
            assert np.array_equal(cls, ref), (s, k, np.nonzero(cls != ref)[0][:5])
            checked += 1
    assert checked > 20
    g.close(); tok.close()


@pytest.mark.gpu
@pytest.mark.parametrize("static_fill", [False, True])
def test_gpu_counted_repetitions_with_a_just_in_time_cache(static_fill):
    """Entries of counted records are built on first visit like any other; until then the mask comes from the walk of
    the whole vocabulary against the chart, counts included.  Also through the allocation-free fill."""
    from test_jit import _drive
    w = inputs.make_workload("R1024", batch=4, steps=150, vocab_size=8192)
    s, final, _, stats = _drive(w, 6, "each", static_fill=static_fill)
    assert final["n_built"] > 0 and sum(x["n_states"] for x in stats) < 4 * 1200
    s.close()


@pytest.mark.gpu
def test_gpu_counted_repetitions_at_the_full_vocabulary():
    """R1024 as bench.py runs it (16 requests, 128 256 tokens, 256 steps): every step of one request and every
    thirty-second step of all of them against the grammar-text oracle."""
    from test_gpu_parity import _run_trajectories
    w = inputs.make_workload("R1024")
    assert w.vocab.size == 128256 and w.batch == 16
    compared = _run_trajectories(w, set(range(0, w.steps, 32)), check_requests={11})
    assert compared >= w.steps
