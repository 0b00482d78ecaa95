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
    import torch
    tokens = [s.encode() for n in (1, 2, 3) for s in map("".join, itertools.product(alphabet, repeat=n))]
    tokens.append(b"")
    eos = len(tokens) - 1
    tokens += [b"\xf0\x9f" + bytes([65 + i]) for i in range(-len(tokens) % 32)]       # padding that no grammar here accepts
    tok = B.Tokenizer(tokens, eos)
    g = B.Grammar(tok, "ebnf", ebnf, inline_max_states=inline)
    jit = B.Grammar(tok, "ebnf", ebnf, inline_max_states=inline, jit=True)           # nothing built: whole-vocabulary walks
    ov = O.Vocab(tokens, eos)
    og = O.Grammar(ebnf)
    matchers = [B.Matcher(g), B.Matcher(jit)]
    batch = B.Batch(matchers)
    mask = torch.zeros((2, tok.words), dtype=torch.int32, device="cuda")
    st = torch.zeros(2, dtype=torch.int32, device="cuda")
    ids = torch.zeros(2, dtype=torch.int32, device="cuda")
    single = {bytes([ord(c)]): tokens.index(bytes([ord(c)])) for c in alphabet}
    checked = 0
    for prefix in all_strings(alphabet, 4):
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
