"""Parity at the full sizes of the five configs, in the launch configuration bench.py times
(whole batch, full vocabulary, eager calls of the same entry points).

C1 and C2 are compared with the oracle on every step (C1 in test_gpu_parity.py).  For C3-C5 the
oracle's whole-vocabulary masks are compared on a seeded set of (request, step) pairs fixed here:

  C3  every step of 8 seeded requests, and 8 seeded steps of all 128 requests;
  C4  for 8 seeded requests every step inside a tool call plus 16 seeded free-text steps, and 8
      seeded steps of all 64 requests;
  C5  every step of 4 seeded requests, and 4 seeded steps of all 256 requests.

On every (request, step) pair the size-independent properties are checked: the sampled token is
allowed, statuses are OK, EOS terminates.  At the steps where all requests are compared the masks
must also be prefix-closed (an allowed token's longest proper prefix in the vocabulary is allowed)
and the masked logits of the whole batch are compared with the oracle's apply; on the other
sampled steps the masked logits of the sampled rows are compared through row_indices.
"""
import numpy as np
import pytest

from oracle import oracle as O
from oracle import schema_ebnf as SE
from paper_2601_04426_b200 import inputs

pytestmark = pytest.mark.gpu


def _pick(rng, n, k):
    pool = list(range(n))
    return sorted(pool.pop(rng.below(len(pool))) for _ in range(min(k, n)))


def _inside_tool_call(w, b):
    """For every step of request b: does the text before the step's token end inside a tool call
    (after a whole '<tool_call>' and before the end of the matching '</tool_call>')?"""
    out, text = [], b""
    for tok in w.trajectories[b]:
        out.append(text.rfind(b"<tool_call>") > text.rfind(b"</tool_call>"))
        text = b"" if tok == w.vocab.eos_id else text + w.vocab.tokens[tok]
    return out


def sampled_pairs(w):
    """The (request, step) pairs whose masks are compared with the oracle, and the steps at which all are."""
    n, steps, name = w.batch, w.steps, w.name
    rng = inputs.Rng(inputs.config_seed(name) ^ 0x5A3B1E)
    if name == "C2":
        return {0: set(range(steps))}, []
    n_req, n_steps = {"C3": (8, 8), "C4": (8, 8), "C5": (4, 4)}[name]
    reqs, all_steps = _pick(rng, n, n_req), _pick(rng, steps, n_steps)
    wanted = {b: set(all_steps) for b in range(n)}
    for b in reqs:
        if name == "C4":
            inside = _inside_tool_call(w, b)
            free = [t for t in range(steps) if not inside[t]]
            wanted[b] |= {t for t in range(steps) if inside[t]} | {free[i] for i in _pick(rng, len(free), 16)}
        else:
            wanted[b] |= set(range(steps))
    return wanted, all_steps


def _prefix_parent(tokens):
    """parent[t] = id of a token whose bytes are the longest proper prefix of token t's, or -1."""
    ids = {}
    for i, t in enumerate(tokens):
        if t:
            ids.setdefault(t, i)
    parent = np.full(len(tokens), -1, dtype=np.int64)
    for i, t in enumerate(tokens):
        for k in range(len(t) - 1, 0, -1):
            j = ids.get(t[:k])
            if j is not None:
                parent[i] = j
                break
    return parent


@pytest.mark.parametrize("name", ["C2", "C3", "C4", "C5"])
def test_full_size_sampled_parity(name):
    import torch
    from paper_2601_04426_b200 import engine
    w = inputs.make_workload(name)
    steps, n = w.steps, w.batch
    wanted, all_steps = sampled_pairs(w)
    s = engine.Session(w)
    ov = O.Vocab(w.vocab.tokens, w.vocab.eos_id, w.vocab.special_ids)
    og = [O.Grammar(SE.grammar_text(g.kind, g.text)) for g in w.grammars]
    oms = {b: O.Matcher(og[w.request_grammar[b]]) for b in wanted}
    logits_np = inputs.make_logits(w.logits_seed, 1, w.vocab.size, w.dtype)
    raw = (lambda a: a.view(np.uint32)) if w.dtype == "f32" else (lambda a: a)
    parent = _prefix_parent(w.vocab.tokens)
    has_parent = np.nonzero(parent >= 0)[0]
    special = set(w.vocab.special_ids)
    compared, in_call = 0, 0
    try:
        for step in range(steps):
            s.fill()
            mask = s.mask_numpy()
            assert (s.status.cpu().numpy() == 0).all(), step
            toks = np.asarray([w.trajectories[b][step] for b in range(n)])
            assert ((mask[np.arange(n), toks >> 5] >> (toks & 31)) & 1).all(), step      # every sampled token is allowed
            rows_here = [b for b in sorted(oms) if step in wanted[b]]
            for b in rows_here:
                ref = oms[b].mask(ov)
                if not np.array_equal(mask[b], ref):
                    diff = np.nonzero(O.unpack_bits(mask[b] ^ ref, ov.size))[0]
                    raise AssertionError("%s request %d step %d: %d tokens differ, e.g. %r" % (name, b, step, len(diff), [w.vocab.tokens[t] for t in diff[:8]]))
                compared += 1
            if step in all_steps:
                bits = np.unpackbits(mask.view(np.uint8), axis=1, bitorder="little")[:, :ov.size]
                assert (bits[:, parent[has_parent]] >= bits[:, has_parent]).all(), step          # prefix closure
                assert not bits[:, sorted(special)].any()
                lg = engine.logits_tensor(np.repeat(logits_np, n, axis=0), s.device)
                s.apply(lg)
                assert np.array_equal(raw(engine.logits_numpy(lg)), raw(O.apply_mask(np.repeat(logits_np, n, axis=0), mask))), (name, step)
            elif rows_here and (name == "C2" or step % 8 == 0):
                # masked logits of the sampled rows, through row_indices (the other rows stay untouched)
                lg = engine.logits_tensor(np.repeat(logits_np, n, axis=0), s.device)
                s.apply(lg, torch.tensor(rows_here, dtype=torch.int32, device=s.device))
                got = engine.logits_numpy(lg)
                for b in rows_here:
                    assert np.array_equal(raw(got[b:b + 1]), raw(O.apply_mask(logits_np, mask[b:b + 1]))), (name, b, step)
                for b in [b for b in range(n) if b not in rows_here][:3]:
                    assert np.array_equal(raw(got[b:b + 1]), raw(logits_np))
            s.accept(toks.tolist())
            assert (s.accept_status.cpu().numpy() == 0).all(), step
            for b in range(n):
                if toks[b] == w.vocab.eos_id:
                    assert s.matchers[b].is_terminated()
                    s.reset(b)
            for b, om in oms.items():
                if om.accept_token(ov, int(toks[b])) == 2:
                    om.reset()
        assert compared == sum(len(v) for v in wanted.values())
        if name == "C2":
            assert compared == steps
        elif name == "C3":
            assert compared == 8 * steps + 8 * (n - 8)
        elif name == "C5":
            assert compared == 4 * steps + 4 * (n - 4)
        else:
            assert compared > 8 * 16 + 8 * n
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
