"""Pins for the oracle's token mask, TagDispatch, schema lowering and mask application."""
import json
import os
import re

import numpy as np
import pytest

from oracle import oracle as O
from oracle import schema_ebnf as SE
from paper_2601_04426_b200 import inputs
from golden_util import GOLDEN, load_mask_fixture
from test_oracle_earley import all_strings


@pytest.mark.parametrize("fixture", ["mask_ab_ac.txt", "mask_bool_object.txt", "mask_nested_arrays.txt"])
def test_hand_worked_masks(fixture):
    ebnf, tokens, cases = load_mask_fixture(fixture)
    g = O.Grammar(ebnf)
    eos = tokens.index("")
    v = O.Vocab([t.encode() for t in tokens], eos_id=eos)
    for prefix, allowed in cases:
        m = O.Matcher(g)
        assert m.accept_bytes(prefix.encode()), prefix
        bits = O.unpack_bits(m.mask(v, threads=1), len(tokens))
        got = sorted(tokens[i] for i in range(len(tokens)) if bits[i])
        assert got == sorted(allowed), (prefix, got)


def _small_vocab(seed, size=1024):
    return inputs.make_vocab(seed, size, 8, 3.0)


def test_mask_prefix_closure_and_trajectory_invariants():
    """Allowed tokens are prefix-closed; every token of a valid output is allowed at its step."""
    w = inputs.make_workload("C1", vocab_size=2048)
    vocab = w.vocab
    ov = O.Vocab(vocab.tokens, vocab.eos_id, vocab.special_ids)
    g = O.Grammar(SE.grammar_text(w.grammars[0].kind, w.grammars[0].text))
    m = O.Matcher(g)
    by_bytes = {t: i for i, t in enumerate(vocab.tokens)}
    for step, tok in enumerate(w.trajectories[0]):
        bits = O.unpack_bits(m.mask(ov), vocab.size)
        assert bits[tok], (step, vocab.tokens[tok])
        assert not any(bits[s] for s in vocab.special_ids)
        for tid in np.nonzero(bits)[0]:
            t = vocab.tokens[tid]
            for k in range(1, len(t)):
                pid = by_bytes.get(t[:k])
                if pid is not None:
                    assert bits[pid], (t, t[:k])
        # the mask agrees with whole-string acceptance of each single byte
        for b in (0x22, 0x7B, 0x7D, 0x30, 0x61, 0x20):
            probe = O.Matcher(g)
            probe.accept_bytes(b"".join(vocab.tokens[t] for t in _doc_tokens(w.trajectories[0], step, vocab.eos_id)))
            assert bits[b] == probe.accept_bytes(bytes([b]))
        r = m.accept_token(ov, tok)
        if tok == vocab.eos_id:
            assert r == 2 and m.is_terminated()
            assert m.mask(ov).sum() == 0
            m.reset()
        else:
            assert r == 1


def _doc_tokens(traj, step, eos):
    """Tokens of the current document before `step` (documents are separated by EOS)."""
    start = 0
    for i in range(step):
        if traj[i] == eos:
            start = i + 1
    return traj[start:step]


def test_eos_only_when_root_complete_and_duplicates_agree():
    g = O.Grammar('root ::= "a" "b"?')
    v = O.Vocab([b"a", b"b", b"ab", b"a", b""], eos_id=4)
    m = O.Matcher(g)
    assert list(O.unpack_bits(m.mask(v), 5)) == [True, False, True, True, False]
    m.accept_token(v, 0)
    assert list(O.unpack_bits(m.mask(v), 5)) == [False, True, False, False, True]
    assert m.accept_token(v, 0) == 0 and m.num_sets() == 2          # refused: state unchanged
    assert m.accept_token(v, 4) == 2 and m.accept_token(v, 1) == 0


# ---------------------------------------------------------------------------------------
# TagDispatch (Section 3.2)
# ---------------------------------------------------------------------------------------

def test_tagdispatch_equals_plain_ebnf_lowering():
    """One rule per automaton node, one reference per transition (Section 4.1's construction),
    written by hand for the tag "ab" over the alphabet {a, b, x}."""
    td = O.Grammar('root ::= TagDispatch(("ab", g))\ng ::= "x" "x"?')
    plain = O.Grammar('''
        root ::= n0
        n0 ::= "" | "a" n1 | [bx] n0
        n1 ::= "" | "a" n1 | "b" g n0 | "x" n0
        g ::= "x" "x"?
    ''')
    for s in all_strings("abx", 7):
        assert O.accepts(td, s.encode()) == O.accepts(plain, s.encode()), s
        assert O.is_prefix(td, s.encode()) == O.is_prefix(plain, s.encode()), s


def test_tagdispatch_with_stop_string_equals_plain_lowering():
    td = O.Grammar('root ::= TagDispatch(("ab", g), stop_strs=("xb")) "!"\ng ::= "a"')
    # nodes: n0 (nothing), na ("a"), nx ("x"); "ab" -> g then n0; "xb" -> done
    plain = O.Grammar('''
        root ::= n0 "!"
        n0 ::= "a" na | "x" nx | "b" n0 | "!" n0
        na ::= "a" na | "b" g n0 | "x" nx | "!" n0
        nx ::= "a" na | "b" | "x" nx | "!" n0
        g ::= "a"
    ''')
    for s in all_strings("abx!", 6):
        assert O.accepts(td, s.encode()) == O.accepts(plain, s.encode()), s
        assert O.is_prefix(td, s.encode()) == O.is_prefix(plain, s.encode()), s


def test_text_channel_is_free_text_up_to_its_first_stop_string():
    """A TagDispatch without tags (a text channel): accepts exactly the strings that end with a stop
    string and hold no earlier occurrence of one; checked with str.find and with the plain lowering."""
    td = O.Grammar('root ::= TagDispatch(stop_strs=("ab", "bb"))')
    plain = O.Grammar("""
        root ::= n0
        n0 ::= "a" na | "b" nb | "x" n0
        na ::= "a" na | "b" | "x" n0
        nb ::= "a" na | "b" | "x" n0
    """)
    for s in all_strings("abx", 7):
        ends = [s.find(p) + 2 for p in ("ab", "bb") if s.find(p) >= 0]
        member = bool(ends) and min(ends) == len(s)
        assert O.accepts(td, s.encode()) == member == O.accepts(plain, s.encode()), s
        assert O.is_prefix(td, s.encode()) == (not ends or min(ends) == len(s)) == O.is_prefix(plain, s.encode()), s


def test_channel_protocol_lowering_accepts_generated_text():
    rng = inputs.Rng(9)
    tools = inputs.make_tool_set(rng, 4)
    g = O.Grammar(SE.tag_dispatch_to_ebnf(json.dumps(inputs.channel_spec(tools))))
    for _ in range(8):
        text = inputs.sample_channel_text(rng, tools, rng.randint(1, 4)).encode()
        m = O.Matcher(g)
        assert m.accept_bytes(text) and m.can_terminate()
        assert not O.is_prefix(g, text + b"x")                        # the final marker ends the response
        m2 = O.Matcher(g)
        assert m2.accept_bytes(text[:-len(inputs.CH_RETURN)]) and not m2.can_terminate()
        if b"commentary" in text:                                     # inside a tool channel only the arguments grammar applies
            at = text.index(b"<|message|>", text.index(b"commentary")) + len(b"<|message|>")
            assert O.is_prefix(g, text[:at] + b"{") and not O.is_prefix(g, text[:at] + b"x")
        at = text.index(b"analysis<|message|>") + len(b"analysis<|message|>") if b"analysis" in text else None
        if at:                                                        # a text channel takes anything, tags included, up to its end marker
            assert O.is_prefix(g, text[:at] + b"<|channel|>final<|message|>{ x")


def test_tagdispatch_fires_at_earliest_ending_tag():
    tags = ["<a>", "<bc>", "<<b>"]
    g = O.Grammar('root ::= TagDispatch(("<a>", r0), ("<bc>", r1), ("<<b>", r2))\nr0 ::= "0"\nr1 ::= "1"\nr2 ::= "2"')
    rng = inputs.Rng(5)
    alphabet = "<>abc x"
    fired = 0
    for _ in range(400):
        pieces = list(alphabet) + tags + ["<", "<<", "<b", "<a", "<<b", "b>", "c>"]
        text = "".join(pieces[rng.below(len(pieces))] for _ in range(rng.randint(0, 8)))
        ends = [(text.find(t) + len(t), i) for i, t in enumerate(tags) if t in text]
        m = O.Matcher(g)
        if not ends:
            assert m.accept_bytes(text.encode()) and m.can_terminate()
            continue
        end, which = min(ends)
        fired += 1
        assert m.accept_bytes(text[:end].encode())
        assert not m.can_terminate()                      # inside the dispatched grammar
        for d in "012":
            probe = O.Matcher(g)
            probe.accept_bytes(text[:end].encode())
            assert probe.accept_bytes(d.encode()) == (d == str(which)), (text, d)
    assert fired > 50


def test_tagdispatch_paper_snippet():
    snippet = open(os.path.join(GOLDEN, "tagdispatch_snippet.txt"), encoding="utf-8").read().rstrip("\n")
    body = inputs.ANY_JSON_EBNF.replace("root    ::= ws value ws", "args    ::= object \" </function>\"")
    g = O.Grammar('root ::= TagDispatch(("<function=get_weather>", args))\n' + body)
    m = O.Matcher(g)
    assert m.accept_bytes(snippet.encode()) and m.can_terminate()
    cut = snippet.index("{") + 5
    m2 = O.Matcher(g)
    assert m2.accept_bytes(snippet[:cut].encode()) and not m2.can_terminate()
    assert not O.is_prefix(g, snippet.replace('{"city"', '{city').encode())


# ---------------------------------------------------------------------------------------
# schema lowering, checked at the level of languages
# ---------------------------------------------------------------------------------------

def _validate(schema, value, defs):
    """Independent semantic check of a parsed JSON value against the schema subset."""
    if "$ref" in schema:
        return _validate(defs[schema["$ref"].rsplit("/", 1)[1]], value, defs)
    if "enum" in schema:
        return value in schema["enum"] and not isinstance(value, bool) or (isinstance(value, bool) and value in schema["enum"])
    t = schema["type"]
    if t == "object":
        return (isinstance(value, dict) and list(value) == list(schema["properties"])
                and all(_validate(s, value[k], defs) for k, s in schema["properties"].items()))
    if t == "array":
        return (isinstance(value, list) and schema.get("minItems", 0) <= len(value)
                and ("maxItems" not in schema or len(value) <= schema["maxItems"])
                and all(_validate(schema["items"], x, defs) for x in value))
    if t == "string":
        return (isinstance(value, str) and schema.get("minLength", 0) <= len(value)
                and ("maxLength" not in schema or len(value) <= schema["maxLength"]))
    if t == "integer":
        return isinstance(value, int) and not isinstance(value, bool)
    if t == "number":
        return isinstance(value, (int, float)) and not isinstance(value, bool)
    if t == "boolean":
        return isinstance(value, bool)
    if t == "null":
        return value is None
    raise ValueError(t)


def test_schema_lowering_language():
    rng = inputs.Rng(99)
    shared = {"pt": {"type": "object", "properties": {"x": {"type": "number"}, "y": {"type": "integer"}}, "required": ["x", "y"]}}
    alphabet = b'{}[]:,"\\ -.0123456789etrufalsn'
    accepted_mutants = 0
    for case in range(12):
        schema = inputs.make_object_schema(rng, rng.randint(2, 7), 3, shared=shared, shared_share=0.2)
        schema["$defs"] = shared
        g = O.Grammar(SE.schema_to_ebnf(json.dumps(schema)))
        for _ in range(8):
            doc = inputs.sample_document(schema, rng, wide=True).encode("utf-8")
            assert _validate(schema, json.loads(doc), shared)
            m = O.Matcher(g)
            assert m.accept_bytes(doc) and m.can_terminate(), doc
            assert not O.accepts(g, doc[:-1])
            for _ in range(10):
                pos = rng.below(len(doc))
                b = bytes([alphabet[rng.below(len(alphabet))]])
                kind = rng.below(3)
                mut = doc[:pos] + b + doc[pos + 1:] if kind == 0 else (doc[:pos] + doc[pos + 1:] if kind == 1 else doc[:pos] + b + doc[pos:])
                if O.accepts(g, mut):
                    accepted_mutants += 1
                    assert _validate(schema, json.loads(mut), shared), mut
                    # the fixed layout: separators are exactly ", " and ": " outside strings
                    assert re.sub(r'"(?:[^"\\]|\\.)*"', '""', mut.decode()).count(",") == re.sub(r'"(?:[^"\\]|\\.)*"', '""', mut.decode()).count(", ")
    assert accepted_mutants > 10


def test_schema_bounds_exact():
    g = O.Grammar(SE.schema_to_ebnf(json.dumps({"type": "string", "minLength": 2, "maxLength": 4})))
    for n in range(7):
        assert O.accepts(g, b'"' + b"a" * n + b'"') == (2 <= n <= 4)
    assert O.accepts(g, '"é\\n😀"'.encode()) and not O.accepts(g, b'"a\\x"')
    g = O.Grammar(SE.schema_to_ebnf(json.dumps({"type": "array", "items": {"type": "boolean"}, "minItems": 1, "maxItems": 3})))
    for n in range(6):
        assert O.accepts(g, ("[" + ", ".join(["true"] * n) + "]").encode()) == (1 <= n <= 3)
    g = O.Grammar(SE.schema_to_ebnf(json.dumps({"type": "array", "items": {"type": "integer"}})))
    for n in range(5):
        assert O.accepts(g, ("[" + ", ".join(["-7"] * n) + "]").encode())
    g = O.Grammar(SE.schema_to_ebnf(json.dumps({"type": "number"})))
    for s, ok in [("0", 1), ("-0", 1), ("01", 0), ("1.5e-3", 1), ("1.", 0), (".5", 0), ("1e", 0), ("-", 0), ("12E+4", 1)]:
        assert O.accepts(g, s.encode()) == bool(ok), s
    with pytest.raises(ValueError):
        SE.schema_to_ebnf(json.dumps({"type": "object", "properties": {"a": {"type": "string", "pattern": "x"}}, "required": []}))


def test_tag_dispatch_spec_lowering_accepts_generated_text():
    rng = inputs.Rng(4)
    tools = inputs.make_tool_set(rng, 5)
    spec = inputs.tag_dispatch_spec(tools)
    g = O.Grammar(SE.tag_dispatch_to_ebnf(json.dumps(spec)))
    for _ in range(10):
        text = inputs.sample_tool_text(rng, tools, "<tool_call>", "</tool_call>", rng.randint(1, 3), 60).encode()
        m = O.Matcher(g)
        assert m.accept_bytes(text) and m.can_terminate()
        inside = text.index(b"<tool_call>") + len(b"<tool_call>") + 3
        m2 = O.Matcher(g)
        assert m2.accept_bytes(text[:inside]) and not m2.can_terminate()
        assert not O.is_prefix(g, text[:inside - 3] + b"x")


# ---------------------------------------------------------------------------------------
# mask application (Section 2.1)
# ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_apply_closed_form(dtype):
    rows, vocab = 3, 1000
    logits = inputs.make_logits(11, rows, vocab, dtype)
    if dtype == "f32":
        logits[0, 5] = np.nan
        logits[1, 7] = -0.0
    else:
        logits[0, 5] = 0x7FC1
        logits[1, 7] = 0x8000
    bits = inputs.stream_u64(3, rows * vocab).reshape(rows, vocab) % 3 == 0
    bits[0, 5] = False
    bits[1, 7] = True
    words = np.zeros((rows, (vocab + 31) // 32), dtype=np.uint32)
    for r in range(rows):
        packed = np.packbits(np.pad(bits[r], (0, words.shape[1] * 32 - vocab)).astype(np.uint8), bitorder="little")
        words[r] = packed.view(np.uint32)
    out = O.apply_mask(logits, words)
    ninf = np.float32(-np.inf).view(np.uint32) if dtype == "f32" else np.uint16(0xFF80)
    raw_in = logits.view(np.uint32) if dtype == "f32" else logits
    raw_out = out.view(np.uint32) if dtype == "f32" else out
    expect = np.where(bits, raw_in, ninf)
    assert np.array_equal(raw_out, expect)
    assert (raw_out != ninf).sum() == bits.sum()          # popcount = number of surviving logits
