"""Pins for the CPU oracle's recogniser: brute force, library regex, json.loads, UTF-8 decoding.

None of these re-use the oracle's own formulas: membership is decided by an independent
bottom-up language enumeration, by Python's `re`, by `json.loads` or by `bytes.decode`.
"""
import itertools
import json
import re

import pytest

from oracle import oracle as O
from paper_2601_04426_b200 import inputs


def enumerate_language(cfg, root, max_len):
    """All sentences of length <= max_len, by iterating set equations to a fixpoint.

    cfg: {nonterminal: [alternative, ...]}, an alternative is a list of symbols, a symbol is a
    nonterminal name (a key of cfg) or a terminal string.
    """
    lang = {nt: set() for nt in cfg}
    changed = True
    while changed:
        changed = False
        for nt, alts in cfg.items():
            for alt in alts:
                partial = {""}
                for sym in alt:
                    choices = lang[sym] if sym in cfg else {sym}
                    partial = {p + c for p in partial for c in choices if len(p) + len(c) <= max_len}
                    if not partial:
                        break
                new = partial - lang[nt]
                if new:
                    lang[nt] |= new
                    changed = True
    return lang[root]


def all_strings(alphabet, max_len):
    for n in range(max_len + 1):
        for tup in itertools.product(alphabet, repeat=n):
            yield "".join(tup)


CFG_CASES = [
    # (name, EBNF text, hand-written CFG of the same language, alphabet, slack)
    ("dyck", 'root ::= "" | "a" root "b" root',
     {"S": [[], ["a", "S", "b", "S"]]}, "ab", 6),
    ("left_recursive_expr", 'root ::= root "+" term | term\nterm ::= "x" | "(" root ")"',
     {"S": [["S", "+", "T"], ["T"]], "T": [["x"], ["(", "S", ")"]]}, "x+()", 7),
    ("ambiguous", 'root ::= root root | "a" | "b" "c"',
     {"S": [["S", "S"], ["a"], ["b", "c"]]}, "abc", 2),
    ("nullable_chain", 'root ::= opt_b opt_c tail\nopt_b ::= "" | "b"\nopt_c ::= "" | "c"\ntail ::= "" | "a" root',
     {"S": [["B", "C", "T"]], "B": [[], ["b"]], "C": [[], ["c"]], "T": [[], ["a", "S"]]}, "abc", 2),
    ("hidden_left_recursion", 'root ::= n root "a" | "b"\nn ::= ""',
     {"S": [["N", "S", "a"], ["b"]], "N": [[]]}, "ab", 7),
    ("unit_cycle", 'root ::= other | "a"\nother ::= root | "b" root',
     {"S": [["O"], ["a"]], "O": [["S"], ["b", "S"]]}, "ab", 2),
    ("palindromes", 'root ::= "a" root "a" | "b" root "b" | "a" | "b" | ""',
     {"S": [["a", "S", "a"], ["b", "S", "b"], ["a"], ["b"], []]}, "ab", 7),
    ("unproductive_branch", 'root ::= "a" dead | "a" "b"\ndead ::= "c" dead',
     {"S": [["a", "b"]]}, "abc", 2),
]


@pytest.mark.parametrize("name,ebnf,cfg,alphabet,slack", CFG_CASES, ids=[c[0] for c in CFG_CASES])
def test_membership_and_viable_prefix_by_brute_force(name, ebnf, cfg, alphabet, slack):
    g = O.Grammar(ebnf)
    max_len = 6
    lang = enumerate_language(cfg, "S", max_len + slack)
    prefixes = {w[:k] for w in lang for k in range(len(w) + 1)}
    for s in all_strings(alphabet, max_len):
        assert O.accepts(g, s.encode()) == (s in lang), (name, s)
        assert O.is_prefix(g, s.encode()) == (s in prefixes), (name, s)


REGEX_CASES = [
    ('root ::= ("ab" | [c-d])* "a"{1,3} [^a]?', r"(?:ab|[c-d])*a{1,3}[^a]?", "abcd"),
    ('root ::= [ab]+ "c"? ("d" | "dd"){2}', r"[ab]+c?(?:d|dd){2}", "abcd"),
    ('root ::= ("a" | "b"){2,} "c"{0,2}', r"(?:a|b){2,}c{0,2}", "abc"),
    ('root ::= "-"? ("0" | [1-2] [0-2]*) ("." [0-2]+)?', r"-?(?:0|[1-2][0-2]*)(?:\.[0-2]+)?", "-.012"),
    ('root ::= ("a" "b"?)* | "c"{3}', r"(?:ab?)*|c{3}", "abc"),
    ('root ::= [^\\x00-b]{2} ([a-b] | "\\x63")*', r"[^\x00-b]{2}(?:[a-b]|c)*", "abcd"),
]


@pytest.mark.parametrize("ebnf,pattern,alphabet", REGEX_CASES)
def test_regular_grammars_against_python_re(ebnf, pattern, alphabet):
    g = O.Grammar(ebnf)
    rx = re.compile(pattern)
    max_len = 6
    members_long = {s for s in all_strings(alphabet, max_len + 3) if rx.fullmatch(s)}
    prefixes = {w[:k] for w in members_long for k in range(len(w) + 1)}
    for s in all_strings(alphabet, max_len):
        assert O.accepts(g, s.encode()) == (rx.fullmatch(s) is not None), s
        assert O.is_prefix(g, s.encode()) == (s in prefixes), s


def _json_ok(data: bytes) -> bool:
    def bad_constant(_):
        raise ValueError("constant")
    try:
        json.loads(data.decode("utf-8"), parse_constant=bad_constant)
        return True
    except (ValueError, UnicodeDecodeError, RecursionError):
        return False


def test_any_json_grammar_against_json_loads():
    g = O.Grammar(inputs.ANY_JSON_EBNF)
    rng = inputs.Rng(20260104)
    alphabet = b'{}[]:,"\\ \n-.0123456789eEtruefalsn\x01\xc3\xa9ab'
    n_valid = n_corrupt_ok = 0
    for i in range(150):
        doc = inputs.sample_any_json(rng, rng.randint(0, 5)).encode("utf-8")
        assert _json_ok(doc)
        m = O.Matcher(g)
        assert m.accept_bytes(doc) and m.can_terminate(), doc
        n_valid += 1
        # every proper prefix is viable
        for cut in (len(doc) // 3, len(doc) // 2):
            assert O.is_prefix(g, doc[:cut])
        for _ in range(6):                       # one-byte substitutions / deletions / insertions
            pos = rng.below(len(doc))
            b = bytes([alphabet[rng.below(len(alphabet))]])
            kind = rng.below(3)
            mutated = doc[:pos] + b + doc[pos + 1:] if kind == 0 else (doc[:pos] + doc[pos + 1:] if kind == 1 else doc[:pos] + b + doc[pos:])
            assert O.accepts(g, mutated) == _json_ok(mutated), mutated
            n_corrupt_ok += _json_ok(mutated)
    assert n_valid == 150 and n_corrupt_ok > 5      # some mutations stay valid, most do not


def test_any_json_short_strings_exhaustive():
    g = O.Grammar(inputs.ANY_JSON_EBNF)
    alphabet = '[]{}",:1e-. tn'
    for s in all_strings(alphabet, 4):
        assert O.accepts(g, s.encode()) == _json_ok(s.encode()), s


def test_char_class_is_wellformed_utf8():
    g = O.Grammar(r'root ::= [^"\\\x00-\x1f]*')
    good = ["", "abc", "é", "中文", "😀", "߿ࠀ￿\U00010000\U0010ffff", "a\u007fb"]
    for s in good:
        assert O.accepts(g, s.encode("utf-8")), s
    assert not O.accepts(g, b'a"b') and not O.accepts(g, b"a\\") and not O.accepts(g, b"\x1f")
    rng = inputs.Rng(77)
    pool = [0x00, 0x22, 0x41, 0x5C, 0x7F, 0x80, 0xBF, 0xC0, 0xC1, 0xC2, 0xDF, 0xE0, 0xA0, 0x9F, 0xED, 0xEF,
            0xF0, 0x90, 0x8F, 0xF4, 0xF5, 0xFF, 0xE4, 0xB8, 0xAD]
    checked = 0
    for _ in range(6000):
        data = bytes(pool[rng.below(len(pool))] for _ in range(rng.randint(1, 5)))
        try:
            text = data.decode("utf-8")
            expect = not any(c in '"\\' or ord(c) < 0x20 for c in text)
        except UnicodeDecodeError:
            expect = False
        assert O.accepts(g, data) == expect, data
        checked += expect
        # a viable prefix is a prefix of some well-formed string: try every short completion
        viable = False
        tails = [b""] + [bytes(t) for n in (1, 2, 3) for t in itertools.product([0x80, 0x8F, 0x90, 0x9F, 0xA0, 0xBF], repeat=n)]
        for tail in tails:
            try:
                text = (data + tail).decode("utf-8")
            except UnicodeDecodeError:
                continue
            if not any(c in '"\\' or ord(c) < 0x20 for c in text):
                viable = True
                break
        assert O.is_prefix(g, data) == viable, data
    assert checked > 100


def test_class_ranges_with_multibyte_bounds():
    g = O.Grammar('root ::= [a-cà-ÿ一-仿]+')
    assert O.accepts(g, "abcàÿ一".encode())
    assert not O.accepts(g, "d".encode()) and not O.accepts(g, "ß".encode()) and not O.accepts(g, "伀".encode())
    assert O.is_prefix(g, "一".encode()[:2]) and not O.is_prefix(g, "倀".encode()[:2])


def test_grammar_errors():
    for bad in ['root ::= "a', "root ::= [a", "root ::= undefined_rule", "x ::= \"a\"", "root ::= (\"a\"", "root ::= \"a\"{3,2}"]:
        with pytest.raises(ValueError):
            O.Grammar(bad)
