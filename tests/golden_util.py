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
