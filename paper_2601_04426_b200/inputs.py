"""Seeded synthetic inputs: vocabularies, JSON schemas, grammars, documents, trajectories, logits.

This module only *draws inputs*.  It contains no grammar lowering, no parsing and no mask
arithmetic, and it imports neither the CUDA binding nor the CPU oracle, so both sides can
consume byte-identical inputs from it.

Every artefact is a pure function of (config name, base seed).  Randomness comes from one
counter-based generator, splitmix64 (Steele, Lea, Flood 2014: state += 0x9E3779B97F4A7C15,
then two xor-shift-multiply rounds), implemented here once for scalars and once vectorised
with numpy for the large logit tensors.

The five workload shapes stand in for the tool-calling / JSON-schema workloads of the paper's
evaluation (Section 4), whose datasets and tokenizers are not available offline:

  C1  tiny object schema, V=8 192, batch 1, 64 steps, fp32 logits
  C2  20-property depth-3 schema, V=128 256, batch 1, 256 steps, bf16 logits
  C3  128 per-request schemas with shared sub-schemas, V=151 936, batch 128, 128 steps, bf16
  C4  TagDispatch '<tool_call>' -> one of 64 tool schemas, V=128 256, batch 64, 512 steps, fp32
  C5  recursive any-JSON grammar, V=200 064 with UTF-8 tokens, batch 256, 256 steps, bf16
"""
from __future__ import annotations

import json
import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

BASE_SEED = 260104426
_M64 = (1 << 64) - 1
_GAMMA = 0x9E3779B97F4A7C15


def _mix64(z: int) -> int:
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


class Rng:
    """Scalar splitmix64 stream."""

    def __init__(self, seed: int):
        self.state = seed & _M64

    def u64(self) -> int:
        self.state = (self.state + _GAMMA) & _M64
        return _mix64(self.state)

    def below(self, n: int) -> int:
        return self.u64() % n

    def uniform(self) -> float:
        return (self.u64() >> 11) * (1.0 / (1 << 53))

    def choice(self, seq):
        return seq[self.below(len(seq))]

    def randint(self, lo: int, hi: int) -> int:
        """Inclusive bounds."""
        return lo + self.below(hi - lo + 1)

    def fork(self, tag: int) -> "Rng":
        return Rng(_mix64((self.state ^ (tag * _GAMMA)) & _M64))


def stream_u64(seed: int, n: int, start: int = 0) -> np.ndarray:
    """Vectorised splitmix64: element i equals the (start+i+1)-th output of Rng(seed)."""
    idx = np.arange(start + 1, start + n + 1, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = np.uint64(seed & _M64) + idx * np.uint64(_GAMMA)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
    return z


# ----------------------------------------------------------------------------------------
# logits
# ----------------------------------------------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    u = x.astype(np.float32).view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def make_logits(seed: int, rows: int, vocab: int, dtype: str) -> np.ndarray:
    """N(0,1) logits by Box-Muller in fp32.  dtype 'f32' -> float32 array; 'bf16' -> uint16 bits."""
    n = rows * vocab
    half = (n + 1) // 2
    u = stream_u64(seed, 2 * half)
    u1 = ((u[:half] >> np.uint64(40)).astype(np.float32) + np.float32(1.0)) * np.float32(1.0 / (1 << 24))
    u2 = (u[half:] >> np.uint64(40)).astype(np.float32) * np.float32(1.0 / (1 << 24))
    r = np.sqrt(np.float32(-2.0) * np.log(u1)).astype(np.float32)
    ang = (np.float32(2.0 * math.pi) * u2).astype(np.float32)
    z = np.concatenate([r * np.cos(ang), r * np.sin(ang)]).astype(np.float32)[:n].reshape(rows, vocab)
    if dtype == "f32":
        return z
    if dtype == "bf16":
        return f32_to_bf16_bits(z)
    raise ValueError(dtype)


# ----------------------------------------------------------------------------------------
# vocabularies
# ----------------------------------------------------------------------------------------

_ALNUM = b"abcdefghijklmnopqrstuvwxyz0123456789"
_PUNCT = b"{}[]:,\"\\-. \n"
_ALPHABET = _ALNUM + _PUNCT
_LEADERS = b" \n{}[]:,\"-."          # whitespace / punctuation that may lead a token
_UTF8_CHARS = ["é", "ß", "ñ", "ü", "Ω", "и", "中", "文", "日", "本", "한", "€", "→", "😀", "🚀", "𝒱"]
SPECIAL_BYTES = [b"<|pad|>", b"<|bos|>", b"<|unk|>"]


@dataclass
class Vocab:
    tokens: List[bytes]            # index = token id
    eos_id: int
    special_ids: List[int]         # never allowed (EOS is handled separately)

    @property
    def size(self) -> int:
        return len(self.tokens)

    def arena(self) -> Tuple[np.ndarray, np.ndarray]:
        """(bytes uint8[total], offsets int64[V+1]) in token-id order."""
        offs = np.zeros(len(self.tokens) + 1, dtype=np.int64)
        np.cumsum([len(t) for t in self.tokens], out=offs[1:])
        data = np.frombuffer(b"".join(self.tokens), dtype=np.uint8).copy()
        return data, offs


def _length_quotas(n: int, max_len: int, mean_len: float, n_symbols: int, n_fixed_single: int) -> List[int]:
    """How many regular tokens to draw at each byte length 1..max_len.

    A clipped geometric law whose parameter is found by bisection so that the realised mean byte
    length over (single-byte tokens + regular tokens) equals `mean_len`, given that at most 90 %
    of the `n_symbols**L` distinct strings of a short length L can be used (the single-byte
    tokens already exhaust length 1).
    """
    caps = [0] + [int(0.9 * min(n_symbols ** L, 10 ** 12)) for L in range(2, max_len + 1)]

    def quotas(p: float) -> List[float]:
        pmf = [p * (1.0 - p) ** (L - 1) for L in range(1, max_len + 1)]
        pmf[-1] += (1.0 - p) ** max_len
        want = [n * q for q in pmf]
        for _ in range(max_len):
            excess = sum(max(0.0, w - c) for w, c in zip(want, caps))
            if excess <= 1e-9:
                break
            free = [i for i, (w, c) in enumerate(zip(want, caps)) if w < c]
            mass = sum(pmf[i] for i in free)
            want = [min(w, c) for w, c in zip(want, caps)]
            for i in free:
                want[i] += excess * pmf[i] / mass
        return want

    def mean_of(p: float) -> float:
        w = quotas(p)
        return (n_fixed_single + sum((i + 1) * x for i, x in enumerate(w))) / (n_fixed_single + n)

    lo, hi = 1e-3, 0.999            # mean decreases as p grows
    for _ in range(60):
        mid = 0.5 * (lo + hi)
        if mean_of(mid) > mean_len:
            lo = mid
        else:
            hi = mid
    w = quotas(0.5 * (lo + hi))
    out = [int(x) for x in w]
    out[min(max_len, max(2, int(round(mean_len)))) - 1] += n - sum(out)
    return out


def make_vocab(seed: int, size: int, max_len: int, mean_len: float,
               leader_share: float = 0.0, utf8_share: float = 0.0) -> Vocab:
    """Byte-level synthetic vocabulary.

    ids 0..255 are the single bytes; the last id is EOS (empty byte string); the three ids before
    it are special tokens; every other token has a clipped-geometric byte length (calibrated so
    the realised mean is `mean_len`) and bytes drawn from [a-z0-9], JSON punctuation, quote,
    backslash, '-', '.', space and newline.  `leader_share` of the tokens start with
    whitespace/punctuation; `utf8_share` of them contain multi-byte UTF-8 characters, a third of
    those cut in the middle of a character.  Duplicates are re-drawn.
    """
    assert size % 32 == 0 and size > 256 + len(SPECIAL_BYTES) + 1
    rng = Rng(seed)
    tokens: List[bytes] = [bytes([b]) for b in range(256)]
    seen = set(tokens)
    n_regular = size - 1 - len(SPECIAL_BYTES) - 256
    quota = _length_quotas(n_regular, max_len, mean_len, len(_ALPHABET), 256)
    lengths: List[int] = []
    for L, q in enumerate(quota, start=1):
        lengths.extend([L] * q)
    for i in range(len(lengths) - 1, 0, -1):          # seeded Fisher-Yates: ids are not sorted by length
        j = rng.below(i + 1)
        lengths[i], lengths[j] = lengths[j], lengths[i]
    for length in lengths:
        wide = utf8_share > 0.0 and length >= 2 and rng.uniform() < utf8_share
        attempts = 0
        while True:
            attempts += 1
            if wide and attempts <= 64:
                parts: List[bytes] = []
                total = 0
                while total < length + 2:
                    if not parts or rng.uniform() < 0.5:
                        c = rng.choice(_UTF8_CHARS).encode("utf-8")
                    else:
                        c = bytes([_ALPHABET[rng.below(len(_ALPHABET))]])
                    parts.append(c)
                    total += len(c)
                tok = b"".join(parts)
                if rng.below(3) == 0:
                    tok = tok[rng.randint(0, 1):]      # may start inside a character
                tok = tok[:length]                     # may end inside a character
            else:
                bs = bytearray(length)
                for i in range(length):
                    bs[i] = _ALPHABET[rng.below(len(_ALPHABET))]
                if leader_share > 0.0:
                    if rng.uniform() < leader_share:
                        bs[0] = _LEADERS[rng.below(len(_LEADERS))]
                    else:
                        bs[0] = _ALNUM[rng.below(len(_ALNUM))]
                tok = bytes(bs)
            if tok and tok not in seen:
                break
        seen.add(tok)
        tokens.append(tok)
    special_ids = []
    for sb in SPECIAL_BYTES:
        special_ids.append(len(tokens))
        tokens.append(sb)
    eos_id = len(tokens)
    tokens.append(b"")
    assert len(tokens) == size
    return Vocab(tokens=tokens, eos_id=eos_id, special_ids=special_ids)


class GreedyTokenizer:
    """Greedy longest-match tokenisation over a Vocab (always succeeds: single bytes exist)."""

    def __init__(self, vocab: Vocab):
        self.index: Dict[bytes, int] = {}
        special = set(vocab.special_ids) | {vocab.eos_id}
        self.max_len = 1
        for tid, tok in enumerate(vocab.tokens):
            if tid in special or not tok:
                continue
            if tok not in self.index:
                self.index[tok] = tid
                self.max_len = max(self.max_len, len(tok))

    def encode(self, data: bytes) -> List[int]:
        out: List[int] = []
        i, n = 0, len(data)
        while i < n:
            for ln in range(min(self.max_len, n - i), 0, -1):
                tid = self.index.get(data[i:i + ln])
                if tid is not None:
                    out.append(tid)
                    i += ln
                    break
        return out


# ----------------------------------------------------------------------------------------
# JSON schemas (the subset both front ends accept) and documents drawn from schema semantics
# ----------------------------------------------------------------------------------------

_WORD_ALPHA = "abcdefghijklmnopqrstuvwxyz"


def _word(rng: Rng, lo: int = 3, hi: int = 9) -> str:
    return "".join(_WORD_ALPHA[rng.below(26)] for _ in range(rng.randint(lo, hi)))


def _scalar_schema(rng: Rng, kinds: Sequence[str], enum_size: int) -> dict:
    kind = rng.choice(list(kinds))
    if kind == "string":
        cap = rng.choice([None, 8, 16])
        return {"type": "string"} if cap is None else {"type": "string", "maxLength": cap}
    if kind == "enum":
        words: List[str] = []
        while len(words) < enum_size:
            w = _word(rng)
            if w not in words:
                words.append(w)
        return {"enum": words}
    return {"type": kind}


def make_object_schema(rng: Rng, n_props: int, max_depth: int, depth: int = 1,
                       kinds: Sequence[str] = ("string", "integer", "number", "boolean", "enum", "array", "object"),
                       enum_size: int = 8, shared: Optional[Dict[str, dict]] = None,
                       shared_share: float = 0.0) -> dict:
    """Object with `n_props` required properties in declared order, nested to `max_depth`."""
    props: Dict[str, dict] = {}
    while len(props) < n_props:
        key = _word(rng, 3, 10)
        if key in props:
            continue
        if shared and rng.uniform() < shared_share:
            props[key] = {"$ref": "#/$defs/" + rng.choice(sorted(shared))}
            continue
        kind = rng.choice(list(kinds))
        if kind == "object":
            if depth >= max_depth:
                kind = "string"
            else:
                props[key] = make_object_schema(rng, rng.randint(2, 5), max_depth, depth + 1, kinds,
                                                enum_size, shared, shared_share)
                continue
        if kind == "array":
            item = _scalar_schema(rng, ("string", "integer", "number", "boolean"), enum_size)
            props[key] = {"type": "array", "items": item, "maxItems": 5}
            if rng.below(2):
                props[key]["minItems"] = 1
            continue
        props[key] = _scalar_schema(rng, (kind,), enum_size)
    return {"type": "object", "properties": props, "required": list(props)}


_STR_PLAIN = "abcdefghijklmnopqrstuvwxyz0123456789 _-"
_STR_ESCAPES = ["\\n", "\\\"", "\\\\", "\\t", "\\u00e9", "\\/"]
_STR_WIDE = ["é", "中", "😀", "ß"]


def _sample_string_body(rng: Rng, min_len: int, max_len: Optional[int], wide: bool) -> str:
    hi = 12 if max_len is None else max_len
    n = rng.randint(min_len, max(min_len, hi))
    out: List[str] = []
    for _ in range(n):
        r = rng.below(20)
        if r == 0:
            out.append(rng.choice(_STR_ESCAPES))
        elif r == 1 and wide:
            out.append(rng.choice(_STR_WIDE))
        else:
            out.append(_STR_PLAIN[rng.below(len(_STR_PLAIN))])
    return "".join(out)


def _sample_integer(rng: Rng) -> str:
    r = rng.below(6)
    if r == 0:
        return "0"
    digits = rng.randint(1, 6)
    s = str(rng.randint(1, 9)) + "".join(str(rng.below(10)) for _ in range(digits - 1))
    return ("-" if rng.below(4) == 0 else "") + s


def _sample_number(rng: Rng) -> str:
    s = _sample_integer(rng)
    if rng.below(2):
        s += "." + "".join(str(rng.below(10)) for _ in range(rng.randint(1, 4)))
    if rng.below(5) == 0:
        s += rng.choice(["e", "E"]) + rng.choice(["", "+", "-"]) + str(rng.randint(0, 30))
    return s


def sample_document(schema: dict, rng: Rng, defs: Optional[Dict[str, dict]] = None, wide: bool = False) -> str:
    """A JSON text valid for `schema`, in the fixed layout `{"k": v, "k2": v2}` / `[a, b]`."""
    if defs is None:
        defs = schema.get("$defs", {})
    if "$ref" in schema:
        return sample_document(defs[schema["$ref"].rsplit("/", 1)[1]], rng, defs, wide)
    if "enum" in schema:
        return json.dumps(rng.choice(schema["enum"]))
    t = schema["type"]
    if t == "object":
        parts = ['"%s": %s' % (k, sample_document(v, rng, defs, wide)) for k, v in schema["properties"].items()]
        return "{" + ", ".join(parts) + "}"
    if t == "array":
        n = rng.randint(schema.get("minItems", 0), schema.get("maxItems", 4))
        return "[" + ", ".join(sample_document(schema["items"], rng, defs, wide) for _ in range(n)) + "]"
    if t == "string":
        return '"' + _sample_string_body(rng, schema.get("minLength", 0), schema.get("maxLength"), wide) + '"'
    if t == "integer":
        return _sample_integer(rng)
    if t == "number":
        return _sample_number(rng)
    if t == "boolean":
        return rng.choice(["true", "false"])
    if t == "null":
        return "null"
    raise ValueError(t)


# ----------------------------------------------------------------------------------------
# the recursive any-JSON grammar of C5 and documents of a given nesting depth
# ----------------------------------------------------------------------------------------

ANY_JSON_EBNF = r"""
root    ::= ws value ws
value   ::= object | array | string | number | "true" | "false" | "null"
object  ::= "{" ws ( member ( ws "," ws member )* ws )? "}"
member  ::= string ws ":" ws value
array   ::= "[" ws ( value ( ws "," ws value )* ws )? "]"
string  ::= "\"" char* "\""
char    ::= [^"\\\x00-\x1f] | "\\" ( ["\\/bfnrt] | "u" [0-9a-fA-F]{4} )
number  ::= "-"? ( "0" | [1-9] [0-9]* ) ( "." [0-9]+ )? ( [eE] [+\-]? [0-9]+ )?
ws      ::= [ \t\n\r]*
"""


def _ws(rng: Rng) -> str:
    return rng.choice(["", "", "", " ", " ", "\n", "  ", "\n  "])


def sample_any_json(rng: Rng, depth: int, wide: bool = True) -> str:
    """A JSON value whose deepest container nesting is exactly `depth` (depth 0 = scalar)."""
    def scalar() -> str:
        r = rng.below(6)
        if r <= 1:
            return '"' + _sample_string_body(rng, 0, 10, wide) + '"'
        if r == 2:
            return _sample_number(rng)
        if r == 3:
            return _sample_integer(rng)
        return rng.choice(["true", "false", "null"])

    def value(d: int) -> str:
        if d == 0:
            return scalar()
        n = rng.randint(1, 3)
        deep = rng.below(n)
        items = [value(d - 1) if i == deep else value(rng.randint(0, max(0, min(d - 1, 1)))) for i in range(n)]
        if rng.below(2):
            body = ("," + _ws(rng)).join(_ws(rng) + it for it in items)
            return "[" + body + _ws(rng) + "]"
        mem = ['"%s"%s:%s%s' % (_word(rng, 1, 6), _ws(rng), _ws(rng), it) for it in items]
        return "{" + _ws(rng) + ("," + _ws(rng)).join(mem) + _ws(rng) + "}"

    return value(depth)


# ----------------------------------------------------------------------------------------
# TagDispatch workload (C4)
# ----------------------------------------------------------------------------------------

def make_tool_set(rng: Rng, n_tools: int) -> List[dict]:
    tools = []
    names = set()
    while len(tools) < n_tools:
        name = _word(rng, 4, 8) + "_" + _word(rng, 3, 6)
        if name in names:
            continue
        names.add(name)
        schema = make_object_schema(rng, rng.randint(3, 12), 2,
                                    kinds=("string", "integer", "number", "boolean", "enum", "array"),
                                    enum_size=4)
        tools.append({"name": name, "schema": schema})
    return tools


def function_tags_spec(tools: List[dict]) -> dict:
    """One tag per tool: `<function=NAME>` dispatches to that tool's argument object, then `</function>`."""
    return {"tags": [{"tag": "<function=%s>" % t["name"], "end": "</function>", "bare": True, "tools": [t]} for t in tools], "stop_strs": []}


def tag_dispatch_spec(tools: List[dict], tag: str = "<tool_call>", end: str = "</tool_call>") -> dict:
    """One tag that dispatches to `(call_1 | ... | call_n) end`, call_k = {"name": ..., "arguments": ...}."""
    return {"tags": [{"tag": tag, "end": end, "tools": tools}], "stop_strs": []}


def sample_tool_text(rng: Rng, tools: List[dict], tag: str, end: str, n_calls: int, min_tokens_hint: int) -> str:
    """Free text (lowercase words and spaces, never '<') interleaved with `n_calls` tool calls."""
    def free(n_words: int) -> str:
        return " ".join(_word(rng, 2, 8) for _ in range(n_words)) + rng.choice([" ", ". ", "\n"])

    words_total = max(8, min_tokens_hint // 2)
    cuts = sorted(rng.randint(1, words_total - 1) for _ in range(n_calls))
    out: List[str] = []
    prev = 0
    for c in cuts:
        out.append(free(max(1, c - prev)))
        tool = rng.choice(tools)
        args = sample_document(tool["schema"], rng)
        out.append(tag + '{"name": "%s", "arguments": %s}' % (tool["name"], args) + end)
        prev = c
    out.append(free(max(1, words_total - prev)))
    return "".join(out)


# a channelised response protocol: every message names its channel; text channels run to an end marker, tool
# channels carry the arguments of one tool, a final marker ends the response (Sections 1 and 3.2)
CH_START, CH_CHANNEL, CH_MESSAGE, CH_END, CH_CALL, CH_RETURN = "<|start|>assistant", "<|channel|>", "<|message|>", "<|end|>", "<|call|>", "<|return|>"


def channel_spec(tools: List[dict]) -> dict:
    tags = [{"tag": CH_CHANNEL + name + CH_MESSAGE, "text": True, "end": CH_END} for name in ("analysis", "final")]
    tags += [{"tag": "%scommentary to=functions.%s%s" % (CH_CHANNEL, t["name"], CH_MESSAGE), "end": CH_CALL, "bare": True, "tools": [t]} for t in tools]
    return {"tags": tags, "stop_strs": [CH_RETURN]}


def sample_channel_text(rng: Rng, tools: List[dict], n_messages: int) -> str:
    def free(k: int) -> str:
        return " ".join(_word(rng, 2, 8) for _ in range(k)) + rng.choice(["", ".", "\n"])
    out: List[str] = []
    for _ in range(n_messages):
        out.append(CH_START)
        if rng.below(2):
            out.append(CH_CHANNEL + "analysis" + CH_MESSAGE + free(rng.randint(3, 14)) + CH_END)
        else:
            tool = rng.choice(tools)
            out.append("%scommentary to=functions.%s%s%s%s" % (CH_CHANNEL, tool["name"], CH_MESSAGE, sample_document(tool["schema"], rng), CH_CALL))
    out.append(CH_START + CH_CHANNEL + "final" + CH_MESSAGE + free(rng.randint(4, 16)) + CH_END + CH_RETURN)
    return "".join(out)


_tool_pool_cache: List[dict] = []


def _tool_pool() -> List[dict]:
    """The seeded pool of 1 908 tools (the size of the tool pool in Section 4.1) with distinct names."""
    if not _tool_pool_cache:
        _tool_pool_cache.extend(make_function_tags(Rng(BASE_SEED * 10 + 300000), 1908, tag_len=24))
    return _tool_pool_cache


def make_function_tags(rng: Rng, n_tags: int, tag_len: int = 20) -> List[dict]:
    """`n_tags` tools whose tags share the prefix `<function=` and are `tag_len` bytes long in total
    (the shape of the paper's tag-count experiment, Section 4.1), each with a small argument schema."""
    tools, names = [], set()
    body = tag_len - len("<function=") - 1
    while len(tools) < n_tags:
        name = _word(rng, body, body)
        if name in names:
            continue
        names.add(name)
        schema = make_object_schema(rng, rng.randint(1, 4), 1, kinds=("string", "integer", "number", "boolean", "enum"), enum_size=3)
        tools.append({"name": name, "schema": schema})
    return tools


def sample_function_text(rng: Rng, tools: List[dict], n_calls: int, n_words: int) -> str:
    def free(k: int) -> str:
        return " ".join(_word(rng, 2, 8) for _ in range(k)) + rng.choice([" ", ". ", "\n"])
    out = [free(max(1, n_words // (n_calls + 1)))]
    for _ in range(n_calls):
        tool = rng.choice(tools)
        out.append("<function=%s>%s</function>" % (tool["name"], sample_document(tool["schema"], rng)))
        out.append(free(max(1, n_words // (n_calls + 1))))
    return "".join(out)


# ----------------------------------------------------------------------------------------
# configs
# ----------------------------------------------------------------------------------------

@dataclass
class GrammarSpec:
    kind: str                     # "ebnf" | "json_schema" | "tag_dispatch"
    text: str                     # grammar text / schema JSON / TagDispatch spec JSON
    root: str = "root"


@dataclass
class Workload:
    name: str
    vocab: Vocab
    grammars: List[GrammarSpec]                 # distinct grammars
    request_grammar: List[int]                  # request -> index into grammars
    trajectories: List[List[int]]               # request -> token ids, one per step (EOS ends a document)
    documents: List[List[bytes]]                # request -> the documents its trajectory spells
    dtype: str                                  # "f32" | "bf16"
    steps: int
    logits_seed: int
    meta: dict = field(default_factory=dict)

    @property
    def batch(self) -> int:
        return len(self.request_grammar)


_SHAPES = {
    #        V       Lmax mean leaders utf8  batch steps dtype
    "C1": (8192,     12,  3.5, 0.0,    0.0,  1,    64,   "f32"),
    "C2": (128256,   16,  4.0, 0.3,    0.0,  1,    256,  "bf16"),
    "C3": (151936,   16,  4.0, 0.3,    0.0,  128,  128,  "bf16"),
    "C4": (128256,   16,  4.0, 0.3,    0.0,  64,   512,  "f32"),
    "C5": (200064,   24,  4.5, 0.0,    0.1,  256,  256,  "bf16"),
    # many-tag TagDispatch (Section 4.1's tag-count experiment): 5 / 20 / 50 / 100 tags of 20 bytes with a common prefix
    "T5": (128256,   16,  4.0, 0.3,    0.0,  16,   128,  "bf16"),
    "T20": (128256,  16,  4.0, 0.3,    0.0,  16,   128,  "bf16"),
    "T50": (128256,  16,  4.0, 0.3,    0.0,  16,   128,  "bf16"),
    "T100": (128256, 16,  4.0, 0.3,    0.0,  16,   128,  "bf16"),
    # channelised response protocol with 16 / 64 tools (text channels with stop strings, one tool channel per tool)
    "H16": (128256,  16,  4.0, 0.3,    0.0,  32,   256,  "bf16"),
    "H64": (128256,  16,  4.0, 0.3,    0.0,  32,   256,  "bf16"),
    # inter-request dynamism (Section 4.1): every request draws its own subset of 10 / 100 / 500 tools from one pool of
    # 1 908 tools, one `<function=NAME>` tag per tool; what the requests share are the tools' argument grammars
    "P10": (128256,  16,  4.0, 0.3,    0.0,  8,    64,   "bf16"),
    "P100": (128256, 16,  4.0, 0.3,    0.0,  8,    64,   "bf16"),
    "P500": (128256, 16,  4.0, 0.3,    0.0,  8,    64,   "bf16"),
    # long bounded repetitions (Section 3.6: minLength / maxLength / minItems / maxItems in the hundreds to thousands)
    "R256": (128256,  16,  4.0, 0.3,    0.0,  16,   256,  "bf16"),
    "R1024": (128256, 16,  4.0, 0.3,    0.0,  16,   256,  "bf16"),
    "R4096": (128256, 16,  4.0, 0.3,    0.0,  16,   256,  "bf16"),
}

_vocab_cache: Dict[Tuple, Vocab] = {}


def config_seed(name: str) -> int:
    if name[0] == "C":
        return BASE_SEED * 10 + int(name[1])
    return BASE_SEED * 10 + {"T": 1000, "R": 100000, "H": 200000, "P": 300000}[name[0]] + int(name[1:])


def config_vocab(name: str, vocab_size: Optional[int] = None) -> Vocab:
    V, lmax, mean, lead, utf8, _, _, _ = _SHAPES[name]
    if vocab_size is not None:
        V = vocab_size
    # C2 and C4 share one Llama-3-sized vocabulary
    seed_name = "C2" if (name == "C4" or name[0] in "TRHP") else name
    key = (seed_name, V)
    if key not in _vocab_cache:
        _vocab_cache[key] = make_vocab(config_seed(seed_name) ^ 0x5EED, V, lmax, mean, lead, utf8)
    return _vocab_cache[key]


def _trajectory(tok: GreedyTokenizer, eos_id: int, steps: int, doc_source) -> Tuple[List[int], List[bytes]]:
    ids: List[int] = []
    docs: List[bytes] = []
    while len(ids) < steps:
        doc = doc_source()
        docs.append(doc)
        ids.extend(tok.encode(doc))
        ids.append(eos_id)
    return ids[:steps], docs


def make_workload(name: str, batch: Optional[int] = None, steps: Optional[int] = None,
                  vocab_size: Optional[int] = None) -> Workload:
    """Build config `name`.  `batch`, `steps`, `vocab_size` shrink it for tests (same recipe)."""
    V, lmax, mean, lead, utf8, B, S, dtype = _SHAPES[name]
    B = batch if batch is not None else B
    S = steps if steps is not None else S
    vocab = config_vocab(name, vocab_size)
    tok = GreedyTokenizer(vocab)
    seed = config_seed(name)
    rng = Rng(seed)
    grammars: List[GrammarSpec] = []
    request_grammar: List[int] = []
    trajs: List[List[int]] = []
    docs_all: List[List[bytes]] = []
    meta: dict = {}

    if name == "C1":
        r = rng.fork(1)
        words: List[str] = []
        while len(words) < 3:
            w = _word(r)
            if w not in words:
                words.append(w)
        schema = {"type": "object", "properties": {
            _word(r, 3, 8): {"type": "string", "maxLength": 16},
            _word(r, 3, 8): {"type": "integer"},
            _word(r, 3, 8): {"type": "boolean"},
            _word(r, 3, 8): {"enum": words}}}
        schema["required"] = list(schema["properties"])
        grammars.append(GrammarSpec("json_schema", json.dumps(schema)))
        for b in range(B):
            rr = rng.fork(100 + b)
            t, d = _trajectory(tok, vocab.eos_id, S, lambda: sample_document(schema, rr).encode())
            request_grammar.append(0); trajs.append(t); docs_all.append(d)
    elif name == "C2":
        schema = make_object_schema(rng.fork(1), 20, 3)
        grammars.append(GrammarSpec("json_schema", json.dumps(schema)))
        for b in range(B):
            rr = rng.fork(100 + b)
            t, d = _trajectory(tok, vocab.eos_id, S, lambda: sample_document(schema, rr).encode())
            request_grammar.append(0); trajs.append(t); docs_all.append(d)
    elif name == "C3":
        pr = rng.fork(7)
        shared = {"shared_%d" % i: make_object_schema(pr, pr.randint(2, 4), 1,
                                                      kinds=("string", "integer", "number", "boolean", "enum"))
                  for i in range(8)}
        for b in range(B):
            gr = rng.fork(1000 + b)
            schema = make_object_schema(gr, gr.randint(5, 30), gr.randint(1, 3), shared=shared, shared_share=0.1)
            schema["$defs"] = shared
            grammars.append(GrammarSpec("json_schema", json.dumps(schema)))
            rr = rng.fork(5000 + b)
            t, d = _trajectory(tok, vocab.eos_id, S, lambda: sample_document(schema, rr).encode())
            request_grammar.append(b); trajs.append(t); docs_all.append(d)
    elif name == "C4":
        tools = make_tool_set(rng.fork(3), 64)
        spec = tag_dispatch_spec(tools)
        grammars.append(GrammarSpec("tag_dispatch", json.dumps(spec)))
        meta["tools"] = tools
        for b in range(B):
            rr = rng.fork(100 + b)
            n_calls = rr.randint(1, 4)
            t, d = _trajectory(tok, vocab.eos_id, S,
                               lambda: sample_tool_text(rr, tools, "<tool_call>", "</tool_call>", n_calls, S).encode())
            request_grammar.append(0); trajs.append(t); docs_all.append(d)
    elif name == "C5":
        grammars.append(GrammarSpec("ebnf", ANY_JSON_EBNF))
        for b in range(B):
            rr = rng.fork(100 + b)
            depth = rr.randint(1, 16)
            t, d = _trajectory(tok, vocab.eos_id, S, lambda: sample_any_json(rr, depth).encode("utf-8"))
            request_grammar.append(0); trajs.append(t); docs_all.append(d)
            meta.setdefault("depths", []).append(depth)
    elif name[0] == "T":
        tools = make_function_tags(rng.fork(3), int(name[1:]))
        grammars.append(GrammarSpec("tag_dispatch", json.dumps(function_tags_spec(tools))))
        meta["tools"] = tools
        for b in range(B):
            rr = rng.fork(100 + b)
            t, d = _trajectory(tok, vocab.eos_id, S, lambda: sample_function_text(rr, tools, rr.randint(1, 3), 40).encode())
            request_grammar.append(0); trajs.append(t); docs_all.append(d)
    elif name[0] == "P":
        pool_tools = _tool_pool()
        k = int(name[1:])
        for b in range(B):
            sr = rng.fork(50 + b)
            picked = sorted({sr.below(len(pool_tools)) for _ in range(4 * k)})
            sr2 = rng.fork(70 + b)
            while len(picked) > k:
                picked.pop(sr2.below(len(picked)))
            tools = [pool_tools[i] for i in picked]
            grammars.append(GrammarSpec("tag_dispatch", json.dumps(function_tags_spec(tools))))
            rr = rng.fork(100 + b)
            t, d = _trajectory(tok, vocab.eos_id, S, lambda: sample_function_text(rr, tools, rr.randint(1, 3), 30).encode())
            request_grammar.append(b); trajs.append(t); docs_all.append(d)
        meta["pool_size"] = len(pool_tools)
    elif name[0] == "H":
        tools = make_tool_set(rng.fork(3), int(name[1:]))
        grammars.append(GrammarSpec("tag_dispatch", json.dumps(channel_spec(tools))))
        meta["tools"] = tools
        for b in range(B):
            rr = rng.fork(100 + b)
            t, d = _trajectory(tok, vocab.eos_id, S, lambda: sample_channel_text(rr, tools, rr.randint(1, 4)).encode())
            request_grammar.append(0); trajs.append(t); docs_all.append(d)
    elif name[0] == "R":
        # four orderings of one set of bounded properties, so that within the step budget different
        # requests are inside different repetitions; lengths are drawn up to the bounds
        n = int(name[1:])
        r = rng.fork(1)
        props = [
            (_word(r, 3, 8), {"type": "string", "maxLength": n}),
            (_word(r, 3, 8), {"type": "string", "minLength": n // 2, "maxLength": n}),
            (_word(r, 3, 8), {"type": "array", "items": {"type": "integer"}, "maxItems": n // 8}),
            (_word(r, 3, 8), {"type": "array", "items": {"type": "string", "maxLength": 8}, "minItems": n // 16, "maxItems": n // 8}),
        ]
        schemas = []
        for k in range(4):
            order = props[k:] + props[:k]
            schema = {"type": "object", "properties": dict(order), "required": [key for key, _ in order]}
            schemas.append(schema)
            grammars.append(GrammarSpec("json_schema", json.dumps(schema)))
        meta["bound"] = n
        for b in range(B):
            rr = rng.fork(100 + b)
            schema = schemas[b % 4]
            t, d = _trajectory(tok, vocab.eos_id, S, lambda: sample_document(schema, rr).encode())
            request_grammar.append(b % 4); trajs.append(t); docs_all.append(d)
    else:
        raise KeyError(name)
    return Workload(name=name, vocab=vocab, grammars=grammars, request_grammar=request_grammar,
                    trajectories=trajs, documents=docs_all, dtype=dtype, steps=S,
                    logits_seed=seed ^ 0x10617, meta=meta)
