"""CPU oracle -- test infrastructure only: ctypes wrapper over earley_oracle.cpp.

`build()` compiles the C++ file with g++ into oracle/liboracle.so (in tree, git-ignored).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "earley_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-pthread", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        L.orc_grammar_create.restype = vp
        L.orc_grammar_create.argtypes = [C.c_char_p, C.c_char_p, C.c_char_p, C.c_int]
        L.orc_grammar_destroy.argtypes = [vp]
        L.orc_grammar_num_rules.argtypes = [vp]
        L.orc_vocab_create.restype = vp
        L.orc_vocab_create.argtypes = [vp, vp, i32, i32, vp, i32]
        L.orc_vocab_destroy.argtypes = [vp]
        L.orc_matcher_create.restype = vp
        L.orc_matcher_create.argtypes = [vp]
        for name in ("orc_matcher_destroy", "orc_matcher_reset", "orc_matcher_num_sets",
                     "orc_matcher_can_terminate", "orc_matcher_is_terminated"):
            getattr(L, name).argtypes = [vp]
        L.orc_matcher_set_size.argtypes = [vp, C.c_int]
        L.orc_matcher_accept_bytes.argtypes = [vp, C.c_char_p, C.c_int]
        L.orc_matcher_accept_token.argtypes = [vp, vp, i32]
        L.orc_matcher_mask.argtypes = [vp, vp, vp, C.c_int]
        L.orc_apply_f32.argtypes = [vp, i32, i32, i64, vp, i64]
        L.orc_apply_bf16.argtypes = [vp, i32, i32, i64, vp, i64]
        L.orc_tables_create.restype = vp
        L.orc_tables_create.argtypes = [i32, i32, i32, i32, i32] + [vp] * 14
        L.orc_tables_destroy.argtypes = [vp]
        L.orc_tables_classify.argtypes = [vp, vp, i32, i32, vp, C.c_int]
        L.orc_tmatcher_create.restype = vp
        L.orc_tmatcher_create.argtypes = [vp]
        for name in ("orc_tmatcher_destroy", "orc_tmatcher_reset", "orc_tmatcher_can_terminate", "orc_tmatcher_num_sets"):
            getattr(L, name).argtypes = [vp]
        L.orc_tmatcher_accept_bytes.argtypes = [vp, C.c_char_p, C.c_int]
        L.orc_tmatcher_get_set.argtypes = [vp, C.c_int, vp, C.c_int]
        L.orc_tmatcher_get_set_counts.argtypes = [vp, C.c_int, vp, C.c_int]
        L.orc_tmatcher_mask_plain.argtypes = [vp, vp, vp, C.c_int]
        L.orc_tmatcher_mask_merged.argtypes = [vp, vp, vp, vp]
        _lib = L
    return _lib


def default_threads() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


class Grammar:
    def __init__(self, ebnf: str, root: str = "root"):
        err = C.create_string_buffer(512)
        self.h = lib().orc_grammar_create(ebnf.encode("utf-8"), root.encode(), err, 512)
        if not self.h:
            raise ValueError(err.value.decode("utf-8", "replace"))

    def __del__(self):
        if getattr(self, "h", None):
            lib().orc_grammar_destroy(self.h)
            self.h = None


class Vocab:
    """tokens: list of bytes in token-id order."""

    def __init__(self, tokens: Sequence[bytes], eos_id: int = -1, special_ids: Sequence[int] = ()):
        self.size = len(tokens)
        self.tokens = list(tokens)
        self.eos_id = eos_id
        offs = np.zeros(self.size + 1, dtype=np.int64)
        np.cumsum([len(t) for t in tokens], out=offs[1:])
        data = np.frombuffer(b"".join(tokens) + b"\0", dtype=np.uint8).copy()
        sp = np.asarray(list(special_ids), dtype=np.int32)
        self.h = lib().orc_vocab_create(data.ctypes.data, offs.ctypes.data, self.size, eos_id,
                                        sp.ctypes.data if len(sp) else None, len(sp))
        self.words = (self.size + 31) // 32

    def __del__(self):
        if getattr(self, "h", None):
            lib().orc_vocab_destroy(self.h)
            self.h = None


class Matcher:
    def __init__(self, grammar: Grammar):
        self.grammar = grammar
        self.h = lib().orc_matcher_create(grammar.h)

    def __del__(self):
        if getattr(self, "h", None):
            lib().orc_matcher_destroy(self.h)
            self.h = None

    def reset(self):
        lib().orc_matcher_reset(self.h)

    def accept_bytes(self, data: bytes) -> bool:
        return bool(lib().orc_matcher_accept_bytes(self.h, data, len(data)))

    def accept_token(self, vocab: Vocab, token: int) -> int:
        """1 accepted, 0 refused, 2 EOS accepted (terminated)."""
        return lib().orc_matcher_accept_token(self.h, vocab.h, int(token))

    def can_terminate(self) -> bool:
        return bool(lib().orc_matcher_can_terminate(self.h))

    def is_terminated(self) -> bool:
        return bool(lib().orc_matcher_is_terminated(self.h))

    def num_sets(self) -> int:
        return lib().orc_matcher_num_sets(self.h)

    def mask(self, vocab: Vocab, threads: Optional[int] = None) -> np.ndarray:
        out = np.zeros(vocab.words, dtype=np.uint32)
        lib().orc_matcher_mask(self.h, vocab.h, out.ctypes.data, threads or default_threads())
        return out


def accepts(grammar: Grammar, data: bytes) -> bool:
    """Whole-string membership: every byte accepted and the root complete at the end."""
    m = Matcher(grammar)
    return m.accept_bytes(data) and m.can_terminate()


def is_prefix(grammar: Grammar, data: bytes) -> bool:
    return Matcher(grammar).accept_bytes(data)


def apply_mask(logits: np.ndarray, mask_words: np.ndarray) -> np.ndarray:
    """Returns a masked copy.  float32 arrays, or uint16 arrays holding bf16 bit patterns."""
    out = np.ascontiguousarray(logits).copy()
    mask = np.ascontiguousarray(mask_words, dtype=np.uint32)
    rows, vocab = out.shape
    assert mask.shape[0] == rows
    if out.dtype == np.float32:
        lib().orc_apply_f32(out.ctypes.data, rows, vocab, out.shape[1], mask.ctypes.data, mask.shape[1])
    elif out.dtype == np.uint16:
        lib().orc_apply_bf16(out.ctypes.data, rows, vocab, out.shape[1], mask.ctypes.data, mask.shape[1])
    else:
        raise TypeError(out.dtype)
    return out


def unpack_bits(words: np.ndarray, n: int) -> np.ndarray:
    """uint32 words (LSB first) -> bool[n]."""
    b = np.unpackbits(np.ascontiguousarray(words, dtype=np.uint32).view(np.uint8), bitorder="little")
    return b[:n].astype(bool)


class Tables:
    """Flattened grammar tables as exported by a compiler (plain arrays)."""

    FIELDS = ("rule_start", "state_rule", "state_final", "cedge_begin", "cedge_class", "cedge_target",
              "redge_begin", "redge_rule", "redge_target", "class_bits")

    def __init__(self, n_rules: int, n_states: int, n_classes: int, root_rule: int, root_nullable: int, **arrays):
        self.n_rules, self.n_states, self.n_classes = n_rules, n_states, n_classes
        self.root_rule, self.root_nullable = root_rule, root_nullable
        self.a = {}
        for f in self.FIELDS:
            dt = np.uint8 if f == "state_final" else (np.uint32 if f == "class_bits" else np.int32)
            self.a[f] = np.ascontiguousarray(arrays[f], dtype=dt)
        # counted repetitions (Section 3.6): bounds per rule and the edges that start the next iteration; absent or
        # empty when the grammar has none
        self.counted = "rule_rep_hi" in arrays and np.asarray(arrays["rule_rep_hi"]).size > 0
        for f, dt in (("rule_rep_lo", np.int32), ("rule_rep_hi", np.int32), ("cedge_iter", np.uint8), ("redge_iter", np.uint8)):
            self.a[f] = np.ascontiguousarray(arrays[f], dtype=dt) if self.counted else np.zeros(0, dtype=dt)
        if self.counted:       # (an edge array may be empty: pass a valid pointer anyway)
            for f in ("cedge_iter", "redge_iter"):
                if self.a[f].size == 0:
                    self.a[f] = np.zeros(1, dtype=np.uint8)
        ptr = lambda f: self.a[f].ctypes.data if self.a[f].size else None
        self.h = lib().orc_tables_create(n_rules, n_states, n_classes, root_rule, root_nullable,
                                         *[ptr(f) for f in self.FIELDS],
                                         *[ptr(f) for f in ("rule_rep_lo", "rule_rep_hi", "cedge_iter", "redge_iter")])

    def __del__(self):
        if getattr(self, "h", None):
            lib().orc_tables_destroy(self.h)
            self.h = None

    def scannable_states(self) -> List[int]:
        cb = self.a["cedge_begin"]
        return [s for s in range(self.n_states) if cb[s + 1] > cb[s]]

    def classify(self, vocab: Vocab, state: int, threads: Optional[int] = None, count: int = 0) -> np.ndarray:
        """uint8[V]: 1 accepted, 2 uncertain, 0 rejected.  count: iterations finished before the current one, for a
        state of a counted repetition (Section 3.6)."""
        out = np.zeros(vocab.size, dtype=np.uint8)
        lib().orc_tables_classify(self.h, vocab.h, int(state), int(count), out.ctypes.data, threads or default_threads())
        return out


class TableMatcher:
    def __init__(self, tables: Tables):
        self.tables = tables
        self.h = lib().orc_tmatcher_create(tables.h)

    def __del__(self):
        if getattr(self, "h", None):
            lib().orc_tmatcher_destroy(self.h)
            self.h = None

    def reset(self):
        lib().orc_tmatcher_reset(self.h)

    def accept_bytes(self, data: bytes) -> bool:
        return bool(lib().orc_tmatcher_accept_bytes(self.h, data, len(data)))

    def can_terminate(self) -> bool:
        return bool(lib().orc_tmatcher_can_terminate(self.h))

    def num_sets(self) -> int:
        return lib().orc_tmatcher_num_sets(self.h)

    def get_set(self, i: int) -> List[tuple]:
        buf = np.zeros(2 * 4096, dtype=np.int32)
        n = lib().orc_tmatcher_get_set(self.h, i, buf.ctypes.data, 4096)
        return [(int(buf[2 * k]), int(buf[2 * k + 1])) for k in range(min(n, 4096))]

    def get_set_counts(self, i: int) -> List[int]:
        """Iteration counts of the items of set i, in get_set's order."""
        buf = np.zeros(4096, dtype=np.int32)
        n = lib().orc_tmatcher_get_set_counts(self.h, i, buf.ctypes.data, 4096)
        return [int(buf[k]) for k in range(min(n, 4096))]

    def mask_plain(self, vocab: Vocab, threads: Optional[int] = None) -> np.ndarray:
        out = np.zeros(vocab.words, dtype=np.uint32)
        lib().orc_tmatcher_mask_plain(self.h, vocab.h, out.ctypes.data, threads or default_threads())
        return out

    def mask_merged(self, vocab: Vocab):
        out = np.zeros(vocab.words, dtype=np.uint32)
        n = C.c_int64(0)
        lib().orc_tmatcher_mask_merged(self.h, vocab.h, out.ctypes.data, C.byref(n))
        return out, n.value
