"""Reader for the mask fixtures under tests/golden/ (format described in its README)."""
import json
import os

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def load_mask_fixture(name):
    lines = open(os.path.join(GOLDEN, name), encoding="utf-8").read().split("\n")
    assert lines[0].strip() == "grammar:"
    i = 1
    grammar = []
    while lines[i].strip():
        grammar.append(lines[i])
        i += 1
    tokens = None
    cases = []
    for line in lines[i:]:
        line = line.strip()
        if line.startswith("tokens:"):
            tokens = json.loads(line[len("tokens:"):])
        elif line.startswith("after "):
            head, allowed = line[len("after "):].split(" : ", 1)
            cases.append((json.loads(head), json.loads(allowed)))
    return "\n".join(grammar) + "\n", tokens, cases


def load_classify_fixture(name):
    """(grammar text, tokens, [(path, accepted tokens, uncertain tokens)]); the README gives the format."""
    lines = open(os.path.join(GOLDEN, name), encoding="utf-8").read().split("\n")
    assert lines[0].strip() == "grammar:"
    i = 1
    grammar = []
    while lines[i].strip():
        grammar.append(lines[i])
        i += 1
    tokens = None
    cases = []
    for line in lines[i:]:
        line = line.strip()
        if line.startswith("tokens:"):
            tokens = json.loads(line[len("tokens:"):])
        elif line.startswith("state "):
            path, rest = line[len("state "):].split(" : accepted ", 1)
            acc, unc = rest.split(" ; uncertain ", 1)
            cases.append((json.loads(path), json.loads(acc), json.loads(unc)))
    return "\n".join(grammar) + "\n", tokens, cases


def state_at_path(t, path):
    """Follow `path` from the root rule's start state through exported tables `t` (a dict of arrays):
    a string scans its bytes along byte-class edges, "@" crosses the state's only rule reference,
    "@>" enters the rule that reference names (at its start state)."""
    s = int(t["rule_start"][t["root_rule"]])
    for step in path:
        if step in ("@", "@>"):
            b, e = int(t["redge_begin"][s]), int(t["redge_begin"][s + 1])
            assert e - b == 1, (path, step)
            s = int(t["redge_target"][b]) if step == "@" else int(t["rule_start"][t["redge_rule"][b]])
            continue
        for byte in step.encode():
            nxt = [int(t["cedge_target"][e]) for e in range(int(t["cedge_begin"][s]), int(t["cedge_begin"][s + 1]))
                   if (int(t["class_bits"][8 * int(t["cedge_class"][e]) + (byte >> 5)]) >> (byte & 31)) & 1]
            assert len(nxt) == 1, (path, step)
            s = nxt[0]
    return s
