"""Parity at the full sizes of the five configs, in the launch configuration bench.py times
(whole batch, full vocabulary, CUDA-graph-free eager calls of the same entry points).

The oracle needs ~0.1-0.5 s per full-vocabulary mask, so masks are compared on a seeded sample of
(request, step) pairs; on every other pair the size-independent properties are checked: the
sampled token is allowed, statuses are OK, EOS terminates, allowed single-byte tokens agree with
the oracle's byte-level acceptance.  Masked logits are compared on the sampled rows.
"""
import numpy as np
import pytest

from oracle import oracle as O
from oracle import schema_ebnf as SE
from paper_2601_04426_b200 import inputs

pytestmark = pytest.mark.gpu

# (config, steps driven, sampled (request, step) pairs)
CASES = [
    ("C2", 40, [(0, 0), (0, 7), (0, 23), (0, 39)]),
    ("C3", 24, [(0, 0), (5, 3), (17, 9), (64, 15), (127, 23), (99, 20)]),
    ("C4", 40, [(0, 0), (3, 12), (40, 25), (63, 39)]),
    ("C5", 20, [(0, 0), (9, 5), (200, 11), (255, 19), (31, 17)]),
]


@pytest.mark.parametrize("name,steps,sample", CASES, ids=[c[0] for c in CASES])
def test_full_size_sampled_parity(name, steps, sample):
    import torch
    from paper_2601_04426_b200 import engine
    w = inputs.make_workload(name, steps=steps)
    s = engine.Session(w)
    ov = O.Vocab(w.vocab.tokens, w.vocab.eos_id, w.vocab.special_ids)
    wanted = {}
    for b, t in sample:
        wanted.setdefault(b, set()).add(t)
    og = {gi: O.Grammar(SE.grammar_text(w.grammars[gi].kind, w.grammars[gi].text)) for gi in {w.request_grammar[b] for b in wanted}}
    oms = {b: O.Matcher(og[w.request_grammar[b]]) for b in wanted}
    logits_np = inputs.make_logits(w.logits_seed, 1, w.vocab.size, w.dtype)
    n = s.n
    rows = torch.tensor(sorted(wanted), dtype=torch.int32, device=s.device)
    compared = 0
    try:
        for step in range(steps):
            s.fill()
            mask = s.mask_numpy()
            assert (s.status.cpu().numpy() == 0).all(), step
            toks = np.asarray([w.trajectories[b][step] for b in range(n)])
            assert ((mask[np.arange(n), toks >> 5] >> (toks & 31)) & 1).all(), step      # every sampled token is allowed
            for b, om in oms.items():
                if step in wanted[b]:
                    ref = om.mask(ov)
                    assert np.array_equal(mask[b], ref), (name, b, step, int(np.unpackbits((mask[b] ^ ref).view(np.uint8)).sum()))
                    compared += 1
            if any(step in wanted[b] for b in wanted):
                # masked logits of the sampled rows, through row_indices (the other rows stay untouched)
                lg = engine.logits_tensor(np.repeat(logits_np, n, axis=0), s.device)
                s.apply(lg, rows)
                got = engine.logits_numpy(lg)
                raw = (lambda a: a.view(np.uint32)) if w.dtype == "f32" else (lambda a: a)
                for b in wanted:
                    assert np.array_equal(raw(got[b:b + 1]), raw(O.apply_mask(logits_np, mask[b:b + 1]))), (name, b, step)
                untouched = [b for b in range(n) if b not in wanted][:3]
                for b in untouched:
                    assert np.array_equal(raw(got[b:b + 1]), raw(logits_np))
            s.accept(toks.tolist())
            assert (s.accept_status.cpu().numpy() == 0).all(), step
            for b in range(n):
                if toks[b] == w.vocab.eos_id:
                    s.reset(b)
            for b, om in oms.items():
                if om.accept_token(ov, int(toks[b])) == 2:
                    om.reset()
        assert compared == len(sample)
    finally:
        s.close()


def test_vocabulary_too_large_for_one_cluster_takes_the_two_kernel_path():
    """Above 8 x 2048 x 32 = 524 288 tokens a row slice no longer fits the cluster kernel's shared
    memory and the fill runs as merge + check kernels; masks must not change."""
    import torch
    from paper_2601_04426_b200 import engine
    w = inputs.make_workload("C1", steps=6, vocab_size=524288 + 4096)
    s = engine.Session(w)
    ov = O.Vocab(w.vocab.tokens, w.vocab.eos_id, w.vocab.special_ids)
    om = O.Matcher(O.Grammar(SE.grammar_text(w.grammars[0].kind, w.grammars[0].text)))
    try:
        for step, tok in enumerate(w.trajectories[0]):
            s.fill()
            assert np.array_equal(s.mask_numpy()[0], om.mask(ov)), step
            s.accept([tok])
            assert int(s.accept_status.cpu()[0]) == 0
            if om.accept_token(ov, tok) == 2:
                om.reset()
                s.reset(0)
        # the accept-and-fill entry point on this path: accept kernel, then the two fill kernels
        s.reset(0); om.reset()
        for step, tok in enumerate(w.trajectories[0][:4]):
            s.accept_fill([tok], restart_on_eos=True)
            assert int(s.accept_status.cpu()[0]) == 0 and int(s.status.cpu()[0]) == 0
            if om.accept_token(ov, tok) == 2:
                om.reset()
            assert np.array_equal(s.mask_numpy()[0], om.mask(ov)), step
    finally:
        s.close()
