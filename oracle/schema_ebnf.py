"""CPU oracle -- test infrastructure only: JSON schema / TagDispatch spec -> grammar text.

The paper says only that schemas are converted by "a deterministic conversion function"
(appendix "More Explanation of the Hash Algorithm"), and that minLength / maxLength / minItems /
maxItems become repetitions (Section 3.6).  The subset and layout below are this build's reading:

  object   all listed properties, in declared order, all required, nothing else;
           layout  {"k1": v1, "k2": v2}   (", " and ": " exactly);  no properties -> {}
  string   " char{minLength,maxLength} "  with char = any scalar value except ", \\ and C0
           controls, or a JSON escape (\\" \\\\ \\/ \\b \\f \\n \\r \\t \\uXXXX)
  integer  -?(0|[1-9][0-9]*)
  number   integer, optional fraction .[0-9]+, optional exponent [eE][+-]?[0-9]+
  boolean  true | false          null  null
  enum     the JSON serialisations of the listed scalar values
  array    [ ]  or  [item, item, ...]  within minItems / maxItems
  $ref     "#/$defs/<name>"

Anything else raises ValueError.  This file is written independently of the library's own
lowering (C++); agreement between the two is checked at the level of masks and languages.
"""
from __future__ import annotations

import json
from typing import Dict, List

CHAR_RULE = r'''[^"\\\x00-\x1f] | "\\" ( ["\\/bfnrt] | "u" [0-9a-fA-F]{4} )'''
INTEGER = r'''"-"? ( "0" | [1-9] [0-9]* )'''
NUMBER = INTEGER + r''' ( "." [0-9]+ )? ( [eE] [+\-]? [0-9]+ )?'''


def ebnf_quote(text: str) -> str:
    """An EBNF string literal spelling exactly the UTF-8 bytes of `text`."""
    out = []
    for ch in text:
        o = ord(ch)
        if ch == "\\":
            out.append("\\\\")
        elif ch == '"':
            out.append('\\"')
        elif ch == "\n":
            out.append("\\n")
        elif ch == "\r":
            out.append("\\r")
        elif ch == "\t":
            out.append("\\t")
        elif o < 0x20 or o == 0x7F:
            out.append("\\x%02x" % o)
        else:
            out.append(ch)
    return '"' + "".join(out) + '"'


def json_literal(value) -> str:
    """JSON text of a scalar: compact, non-ASCII kept as is."""
    return json.dumps(value, ensure_ascii=False)


class _Lowering:
    def __init__(self, defs: Dict[str, dict], prefix: str):
        self.defs = defs
        self.prefix = prefix
        self.rules: List[str] = []
        self.def_rule: Dict[str, str] = {}
        self.counter = 0
        self.have_char = False

    def fresh(self, hint: str) -> str:
        self.counter += 1
        return "%s%s_%d" % (self.prefix, hint, self.counter)

    def char_rule(self) -> str:
        name = self.prefix + "jchar"
        if not self.have_char:
            self.have_char = True
            self.rules.append("%s ::= %s" % (name, CHAR_RULE))
        return name

    def expr(self, schema: dict) -> str:
        """An EBNF expression (safe to embed in a sequence) for `schema`."""
        if not isinstance(schema, dict):
            raise ValueError("schema must be an object")
        if "$ref" in schema:
            ref = schema["$ref"]
            if not ref.startswith("#/$defs/"):
                raise ValueError("unsupported $ref " + ref)
            name = ref[len("#/$defs/"):]
            if name not in self.defs:
                raise ValueError("unknown $ref " + ref)
            if name not in self.def_rule:
                rule = self.fresh("def")
                self.def_rule[name] = rule
                self.rules.append("%s ::= %s" % (rule, self.expr(self.defs[name])))
            return self.def_rule[name]
        if "enum" in schema:
            vals = schema["enum"]
            if not vals:
                raise ValueError("empty enum")
            for v in vals:
                if isinstance(v, (dict, list)):
                    raise ValueError("enum of non-scalars is unsupported")
            return "( " + " | ".join(ebnf_quote(json_literal(v)) for v in vals) + " )"
        t = schema.get("type")
        if t == "object":
            props = schema.get("properties", {})
            req = schema.get("required", list(props))
            if list(req) != list(props):
                raise ValueError("every property must be required, in declared order")
            if schema.get("additionalProperties", False) not in (False,):
                raise ValueError("additionalProperties is unsupported")
            if not props:
                return '"{}"'
            parts = []
            first = True
            for key, sub in props.items():
                lead = ("{" if first else ", ") + json_literal(key) + ": "
                first = False
                parts.append(ebnf_quote(lead))
                parts.append(self.expr(sub))
            parts.append('"}"')
            rule = self.fresh("obj")
            self.rules.append("%s ::= %s" % (rule, " ".join(parts)))
            return rule
        if t == "array":
            item = self.expr(schema.get("items", None) or _unsupported("array without items"))
            lo = int(schema.get("minItems", 0))
            hi = schema.get("maxItems")
            if hi is not None and int(hi) < lo:
                raise ValueError("maxItems < minItems")
            if hi is not None and int(hi) == 0:
                return '"[]"'
            more_lo = max(lo - 1, 0)
            rep = "{%d,}" % more_lo if hi is None else "{%d,%d}" % (more_lo, int(hi) - 1)
            body = '%s ( ", " %s )%s' % (item, item, rep)
            rule = self.fresh("arr")
            if lo == 0:
                self.rules.append('%s ::= "[" ( %s )? "]"' % (rule, body))
            else:
                self.rules.append('%s ::= "[" %s "]"' % (rule, body))
            return rule
        if t == "string":
            lo = int(schema.get("minLength", 0))
            hi = schema.get("maxLength")
            if hi is not None and int(hi) < lo:
                raise ValueError("maxLength < minLength")
            ch = self.char_rule()
            if hi is None:
                rep = "*" if lo == 0 else "{%d,}" % lo
            else:
                rep = "{%d,%d}" % (lo, int(hi))
            rule = self.fresh("str")
            self.rules.append('%s ::= "\\"" %s%s "\\""' % (rule, ch, rep))
            return rule
        if t == "integer":
            return "( " + INTEGER + " )"
        if t == "number":
            return "( " + NUMBER + " )"
        if t == "boolean":
            return '( "true" | "false" )'
        if t == "null":
            return '"null"'
        raise ValueError("unsupported schema: " + json.dumps(schema)[:80])


def _unsupported(msg: str):
    raise ValueError(msg)


def schema_to_ebnf(schema_text: str, root: str = "root", prefix: str = "") -> str:
    schema = json.loads(schema_text) if isinstance(schema_text, str) else schema_text
    low = _Lowering(schema.get("$defs", {}), prefix)
    body = low.expr(schema)
    return "\n".join(["%s ::= %s" % (root, body)] + low.rules) + "\n"


def tag_dispatch_to_ebnf(spec_text: str, root: str = "root") -> str:
    """{"tags": [{"tag": t, "end": e, "tools": [{"name": n, "schema": s}, ...]}, ...], "stop_strs": [...]}

    Tag t dispatches to  ( call_1 | ... | call_n ) e  with  call_k = {"name": "n_k", "arguments": <s_k>},
    or, when the tag entry has "bare": true, call_k = <s_k> alone.  A tag entry with "text": true has no
    tools: its body is free text that ends with the entry's "end" string.
    """
    spec = json.loads(spec_text) if isinstance(spec_text, str) else spec_text
    rules: List[str] = []
    pairs = []
    for ti, tag in enumerate(spec["tags"]):
        if tag.get("text"):
            # a channel whose body is free text up to its end marker (Section 3.2's stop strings)
            rules.append("tag_%d ::= TagDispatch(stop_strs=(%s))" % (ti, ebnf_quote(tag["end"])))
            pairs.append("(%s, tag_%d)" % (ebnf_quote(tag["tag"]), ti))
            continue
        calls = []
        for ki, tool in enumerate(tag["tools"]):
            prefix = "t%d_%d_" % (ti, ki)
            sub = schema_to_ebnf(tool["schema"], root=prefix + "args", prefix=prefix)
            rules.append(sub.rstrip("\n"))
            if tag.get("bare"):
                rules.append('%scall ::= %sargs' % (prefix, prefix))
            else:
                head = '{"name": %s, "arguments": ' % json_literal(tool["name"])
                rules.append('%scall ::= %s %sargs "}"' % (prefix, ebnf_quote(head), prefix))
            calls.append(prefix + "call")
        rules.append("tag_%d ::= ( %s ) %s" % (ti, " | ".join(calls), ebnf_quote(tag.get("end", ""))))
        pairs.append("(%s, tag_%d)" % (ebnf_quote(tag["tag"]), ti))
    stops = ", ".join(ebnf_quote(s) for s in spec.get("stop_strs", []))
    head = "%s ::= TagDispatch(%s, stop_strs=(%s))" % (root, ", ".join(pairs), stops)
    return "\n".join([head] + rules) + "\n"


def grammar_text(kind: str, text: str) -> str:
    """EBNF text for any of the three grammar kinds."""
    if kind == "ebnf":
        return text
    if kind == "json_schema":
        return schema_to_ebnf(text)
    if kind == "tag_dispatch":
        return tag_dispatch_to_ebnf(text)
    raise ValueError(kind)
