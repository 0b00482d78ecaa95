"""GPU masks on small grammars with every awkward structure -- nullable rules, left and hidden left
recursion, ambiguity, unit cycles, unproductive branches, bounded repetitions -- checked
exhaustively: after every viable prefix of up to four bytes, the mask over all tokens of up to
three bytes must equal the oracle's.  The oracle itself is pinned on these same grammars by brute
force and by Python's `re` (tests/test_oracle_earley.py)."""
import itertools

import numpy as np
import pytest

from oracle import oracle as O
from paper_2601_04426_b200 import binding as B
from test_oracle_earley import CFG_CASES, REGEX_CASES, all_strings

pytestmark = pytest.mark.gpu

CASES = [(c[0], c[1], c[3]) for c in CFG_CASES] + [("regex_%d" % i, c[0], c[2]) for i, c in enumerate(REGEX_CASES)]


@pytest.mark.parametrize("inline", [-1, 0], ids=["inlined", "rules_kept"])
@pytest.mark.parametrize("name,ebnf,alphabet", CASES, ids=[c[0] for c in CASES])
def test_every_prefix_every_token(name, ebnf, alphabet, inline):
    _every_prefix_every_token(name, ebnf, alphabet, 4, inline_max_states=inline)


def _counted_cases():
    from test_counted_repetition import COUNTED_CASES
    return [("counted_%d" % i, c[0], c[1], min(c[2], 6)) for i, c in enumerate(COUNTED_CASES)]


@pytest.mark.parametrize("name,ebnf,alphabet,max_len", _counted_cases(), ids=[c[0] for c in _counted_cases()])
def test_every_prefix_every_token_with_counted_repetitions(name, ebnf, alphabet, max_len):
    """Repetitions of two or more iterations kept as counters (Section 3.6): tokens of up to three bytes cross
    iteration boundaries, both bounds and the end of the rule from every count."""
    _every_prefix_every_token(name, ebnf, alphabet, max_len, repeat_threshold=2)


def _every_prefix_every_token(name, ebnf, alphabet, max_prefix, **compile_kw):
    import torch
    tokens = [s.encode() for n in (1, 2, 3) for s in map("".join, itertools.product(alphabet, repeat=n))]
    tokens.append(b"")
    eos = len(tokens) - 1
    tokens += [b"\xf0\x9f" + bytes([65 + i]) for i in range(-len(tokens) % 32)]       # padding that no grammar here accepts
    tok = B.Tokenizer(tokens, eos)
    g = B.Grammar(tok, "ebnf", ebnf, **compile_kw)
    jit = B.Grammar(tok, "ebnf", ebnf, jit=True, **compile_kw)                       # nothing built: whole-vocabulary walks
    ov = O.Vocab(tokens, eos)
    og = O.Grammar(ebnf)
    matchers = [B.Matcher(g), B.Matcher(jit)]
    batch = B.Batch(matchers)
    mask = torch.zeros((2, tok.words), dtype=torch.int32, device="cuda")
    st = torch.zeros(2, dtype=torch.int32, device="cuda")
    ids = torch.zeros(2, dtype=torch.int32, device="cuda")
    single = {bytes([ord(c)]): tokens.index(bytes([ord(c)])) for c in alphabet}
    checked = 0
    for prefix in all_strings(alphabet, max_prefix):
        data = prefix.encode()
        om = O.Matcher(og)
        if not om.accept_bytes(data):
            continue
        for m in matchers:
            m.reset()
        for byte in data:
            ids[:] = single[bytes([byte])]
            batch.accept_token(ids.data_ptr(), st.data_ptr())
        assert (st.cpu().numpy() == 0).all(), prefix
        batch.fill_next_token_bitmask(mask.data_ptr(), tok.words, st.data_ptr())
        assert (st.cpu().numpy() == 0).all(), prefix
        ref = om.mask(ov)
        got = mask.cpu().numpy().view(np.uint32)
        for row, what in ((0, "cache"), (1, "walk")):
            if not np.array_equal(got[row], ref):
                diff = np.nonzero(O.unpack_bits(got[row] ^ ref, ov.size))[0]
                raise AssertionError("%s after %r (%s): tokens %r" % (name, prefix, what, [tokens[t] for t in diff[:8]]))
        checked += 1
    assert checked >= 3
    for m in matchers:
        m.close()
    g.close(); jit.close(); tok.close()
