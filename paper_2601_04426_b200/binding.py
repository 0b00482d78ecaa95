"""Thin ctypes binding over the C ABI in include/xg.h: argument marshalling only.

Every computation happens inside libxg.so (CUDA kernels + the host grammar front end).  There is
no fallback: if the library is missing or a call fails, an exception is raised.
Device buffers are passed as raw pointers (e.g. torch.Tensor.data_ptr()); torch is only used by
callers for memory and streams, never imported here.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np

from . import build as _build

XG_OK = 0
XG_ERR_INVALID_ARG, XG_ERR_PARSE, XG_ERR_UNSUPPORTED, XG_ERR_OOM, XG_ERR_CUDA = -1, -2, -3, -4, -5
XG_ERR_CAPACITY, XG_ERR_TOKEN_REJECTED, XG_ERR_TERMINATED, XG_ERR_TIMEOUT, XG_ERR_BOUNDS = -6, -7, -8, -9, -10
XG_EBNF, XG_JSON_SCHEMA, XG_TAG_DISPATCH_JSON = 0, 1, 2
XG_F32, XG_BF16 = 0, 1
XG_STORE_ACCEPT_LIST, XG_STORE_REJECT_LIST, XG_STORE_BITSET = 0, 1, 2
KIND_BY_NAME = {"ebnf": XG_EBNF, "json_schema": XG_JSON_SCHEMA, "tag_dispatch": XG_TAG_DISPATCH_JSON}
DTYPE_BY_NAME = {"f32": XG_F32, "bf16": XG_BF16}

EXPORTS = [
    "xg_last_error", "xg_debug_bounds_enabled", "xg_debug_bounds_check", "xg_tokenizer_create", "xg_tokenizer_destroy", "xg_cache_pool_create", "xg_cache_pool_destroy", "xg_cache_pool_set_limit", "xg_cache_pool_reserve", "xg_cache_pool_stats",
    "xg_compile_grammar", "xg_grammar_destroy", "xg_grammar_get_tables", "xg_grammar_get_rule_hashes", "xg_grammar_get_cache_entry", "xg_grammar_record_of", "xg_grammar_get_state_classes", "xg_grammar_stats", "xg_jit_service",
    "xg_matcher_create", "xg_matcher_reset", "xg_matcher_destroy", "xg_matcher_is_terminated", "xg_matcher_next_fill_work",
    "xg_fill_next_token_bitmask", "xg_fill_next_token_bitmask_static", "xg_apply_token_bitmask", "xg_accept_token",
    "xg_accept_token_ex", "xg_accept_token_and_fill_next_bitmask", "xg_fill_and_apply_token_bitmask",
]
XG_STATIC_FILL_MAX_BATCH = 1024


class XgError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("xg status %d: %s" % (status, message))
        self.status = status


class CompileOptions(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("inline_max_states", C.c_int32), ("max_rule_states", C.c_int32), ("build_cache", C.c_int32),
                ("no_state_compression", C.c_int32), ("jit", C.c_int32), ("jit_precompute", C.c_int32), ("jit_arena_bytes", C.c_int64),
                ("count_node_visits", C.c_int32), ("repeat_threshold", C.c_int32), ("repeat_depth", C.c_int32), ("reserved", C.c_int32)]


class FillWork(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_merge", "n_check", "n_missing", "pad")] + \
               [(n, C.c_int64) for n in ("merge_bytes", "check_tokens", "check_bytes", "row_bytes")]


class JitStats(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_built", "n_pool_hits", "n_in_flight", "n_missing")]


class MatcherOptions(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("max_sets", C.c_int32), ("max_items", C.c_int32)]


class PoolStats(C.Structure):
    _fields_ = [("bytes", C.c_int64), ("reserved_bytes", C.c_int64), ("evicted_bytes", C.c_int64), ("evicted_chunks", C.c_int64), ("live_rules", C.c_int32), ("chunks", C.c_int32)]


class GrammarTables(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_rules", "n_states", "n_classes", "n_class_edges", "n_ref_edges", "root_rule", "root_nullable")] + \
               [(n, C.c_void_p) for n in ("rule_start", "state_rule", "state_final", "cedge_begin", "cedge_class", "cedge_target",
                                          "redge_begin", "redge_rule", "redge_target", "class_bits",
                                          "rule_rep_lo", "rule_rep_hi", "cedge_iter", "redge_iter")] + [("n_records", C.c_int32)]


class CacheEntryView(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("state", "kind", "n_accepted", "n_rejected", "n_uncertain", "n_list")] + \
               [(n, C.c_void_p) for n in ("list", "bitset", "uncertain")]


class GrammarStats(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_rules", "n_states", "n_scannable", "n_classes", "n_entries_built", "n_entries_reused")] + \
               [(n, C.c_int64) for n in ("pairs_classified", "total_accepted", "total_rejected", "total_uncertain")] + \
               [("kind_count", C.c_int32 * 3), ("pad", C.c_int32), ("cache_bytes", C.c_int64), ("frontend_ms", C.c_double), ("cache_build_ms", C.c_double), ("total_checked", C.c_int64),
                ("n_entries_shared", C.c_int64), ("classify_ms", C.c_double), ("node_visits", C.c_int64)]


_lib = None


def lib_path() -> str:
    return _build.LIB_DEBUG if os.environ.get("XG_DEBUG_BOUNDS") == "1" else _build.LIB


def debug_bounds_check(stream: int = 0):
    """Raises XgError(XG_ERR_BOUNDS) if a kernel of the bounds-checking build met an index outside its table."""
    _check(lib().xg_debug_bounds_check(stream))


def lib():
    """Load (building first if the sources are newer) libxg.so -- or, with XG_DEBUG_BOUNDS=1 in the environment,
    the bounds-checking variant libxg_dbg.so.  Raises if that is impossible."""
    global _lib
    if _lib is None:
        path = _build.build(debug_bounds=os.environ.get("XG_DEBUG_BOUNDS") == "1")
        L = C.CDLL(path)
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        L.xg_last_error.restype = C.c_char_p
        L.xg_debug_bounds_enabled.restype = i32
        L.xg_debug_bounds_check.argtypes = [vp]
        L.xg_tokenizer_create.argtypes = [vp, vp, i32, i32, vp, i32, vp, C.POINTER(vp)]
        L.xg_tokenizer_destroy.argtypes = [vp]
        L.xg_tokenizer_destroy.restype = None
        L.xg_cache_pool_create.argtypes = [vp, C.POINTER(vp)]
        L.xg_cache_pool_destroy.argtypes = [vp]
        L.xg_cache_pool_destroy.restype = None
        L.xg_cache_pool_set_limit.argtypes = [vp, i64]
        L.xg_cache_pool_reserve.argtypes = [vp, i64]
        L.xg_cache_pool_stats.argtypes = [vp, C.POINTER(PoolStats)]
        L.xg_compile_grammar.argtypes = [vp, vp, C.c_int, C.c_char_p, C.c_size_t, C.c_char_p, C.POINTER(CompileOptions), vp, C.POINTER(vp)]
        L.xg_grammar_destroy.argtypes = [vp]
        L.xg_grammar_destroy.restype = None
        L.xg_grammar_get_tables.argtypes = [vp, C.POINTER(GrammarTables)]
        L.xg_grammar_get_rule_hashes.argtypes = [vp, vp]
        L.xg_grammar_get_cache_entry.argtypes = [vp, i32, C.POINTER(CacheEntryView)]
        L.xg_grammar_get_state_classes.argtypes = [vp, i32, vp]
        L.xg_grammar_record_of.argtypes = [vp, i32, i32, C.POINTER(C.c_int32)]
        L.xg_jit_service.argtypes = [vp, i32, vp, i32, C.POINTER(JitStats)]
        L.xg_grammar_stats.argtypes = [vp, C.POINTER(GrammarStats)]
        L.xg_matcher_create.argtypes = [vp, C.POINTER(MatcherOptions), vp, C.POINTER(vp)]
        L.xg_matcher_reset.argtypes = [vp, vp]
        L.xg_matcher_destroy.argtypes = [vp]
        L.xg_matcher_destroy.restype = None
        L.xg_matcher_is_terminated.argtypes = [vp, vp, C.POINTER(i32)]
        L.xg_matcher_next_fill_work.argtypes = [vp, vp, C.POINTER(FillWork)]
        L.xg_fill_next_token_bitmask.argtypes = [vp, i32, vp, i64, vp, vp]
        L.xg_fill_next_token_bitmask_static.argtypes = [vp, i32, vp, i64, vp, vp]
        L.xg_apply_token_bitmask.argtypes = [vp, C.c_int, i32, i32, i64, vp, i64, vp, i32, vp]
        L.xg_accept_token.argtypes = [vp, i32, vp, vp, vp]
        L.xg_accept_token_ex.argtypes = [vp, i32, vp, vp, i32, vp]
        L.xg_accept_token_and_fill_next_bitmask.argtypes = [vp, i32, vp, vp, i32, vp, i64, vp, vp]
        L.xg_fill_and_apply_token_bitmask.argtypes = [vp, i32, vp, i64, vp, vp, C.c_int, i64, vp]
        _lib = L
    return _lib


def _check(status: int):
    if status != XG_OK:
        raise XgError(status, lib().xg_last_error().decode("utf-8", "replace"))


class Tokenizer:
    def __init__(self, tokens: Sequence[bytes], eos_id: int = -1, special_ids: Sequence[int] = (), stream: int = 0):
        self.size = len(tokens)
        self.words = (self.size + 31) // 32
        self.eos_id = eos_id
        offs = np.zeros(self.size + 1, dtype=np.int64)
        np.cumsum([len(t) for t in tokens], out=offs[1:])
        data = np.frombuffer(b"".join(tokens) + b"\0", dtype=np.uint8).copy()
        sp = np.asarray(list(special_ids), dtype=np.int32)
        h = C.c_void_p()
        _check(lib().xg_tokenizer_create(data.ctypes.data, offs.ctypes.data, self.size, eos_id,
                                         sp.ctypes.data if len(sp) else None, len(sp), stream, C.byref(h)))
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            lib().xg_tokenizer_destroy(self.h)
            self.h = None


class CachePool:
    def __init__(self, tokenizer: Tokenizer):
        h = C.c_void_p()
        _check(lib().xg_cache_pool_create(tokenizer.h, C.byref(h)))
        self.h = h

    def set_limit(self, max_bytes: int):
        _check(lib().xg_cache_pool_set_limit(self.h, int(max_bytes)))

    def reserve(self, n_bytes: int):
        _check(lib().xg_cache_pool_reserve(self.h, int(n_bytes)))

    def stats(self) -> dict:
        s = PoolStats()
        _check(lib().xg_cache_pool_stats(self.h, C.byref(s)))
        return {n: getattr(s, n) for n, _ in PoolStats._fields_}

    def close(self):
        if getattr(self, "h", None):
            lib().xg_cache_pool_destroy(self.h)
            self.h = None


class Grammar:
    def __init__(self, tokenizer: Optional[Tokenizer], kind, text: str, pool: Optional[CachePool] = None, root: Optional[str] = None,
                 inline_max_states: int = -1, build_cache: bool = True, stream: int = 0, state_compression: bool = True,
                 jit: bool = False, jit_precompute: int = 0, jit_arena_bytes: int = 0, count_node_visits: bool = False,
                 repeat_threshold: int = 0, repeat_depth: int = 0):
        kind = KIND_BY_NAME.get(kind, kind)
        raw = text.encode("utf-8") if isinstance(text, str) else text
        opt = CompileOptions(C.sizeof(CompileOptions), inline_max_states, 0, 1 if build_cache else 0, 0 if state_compression else 1,
                             1 if jit else 0, int(jit_precompute), int(jit_arena_bytes), 1 if count_node_visits else 0, int(repeat_threshold), int(repeat_depth), 0)
        h = C.c_void_p()
        _check(lib().xg_compile_grammar(tokenizer.h if tokenizer else None, pool.h if pool else None, kind, raw, len(raw),
                                        root.encode() if root else None, C.byref(opt), stream, C.byref(h)))
        self.h = h
        self.tokenizer = tokenizer

    def close(self):
        if getattr(self, "h", None):
            lib().xg_grammar_destroy(self.h)
            self.h = None

    def tables(self) -> dict:
        """Copies of the flattened tables as numpy arrays plus the scalar fields."""
        t = GrammarTables()
        _check(lib().xg_grammar_get_tables(self.h, C.byref(t)))

        def arr(ptr, n, dt):
            if n == 0 or not ptr:
                return np.zeros(0, dtype=dt)
            return np.ctypeslib.as_array(C.cast(ptr, C.POINTER(np.ctypeslib.as_ctypes_type(dt))), shape=(n,)).copy()
        return dict(
            n_rules=t.n_rules, n_states=t.n_states, n_classes=t.n_classes, root_rule=t.root_rule, root_nullable=t.root_nullable,
            rule_start=arr(t.rule_start, t.n_rules, np.int32), state_rule=arr(t.state_rule, t.n_states, np.int32),
            state_final=arr(t.state_final, t.n_states, np.uint8),
            cedge_begin=arr(t.cedge_begin, t.n_states + 1, np.int32), cedge_class=arr(t.cedge_class, t.n_class_edges, np.int32),
            cedge_target=arr(t.cedge_target, t.n_class_edges, np.int32),
            redge_begin=arr(t.redge_begin, t.n_states + 1, np.int32), redge_rule=arr(t.redge_rule, t.n_ref_edges, np.int32),
            redge_target=arr(t.redge_target, t.n_ref_edges, np.int32), class_bits=arr(t.class_bits, t.n_classes * 8, np.uint32),
            # counted repetitions (empty arrays when the grammar has none)
            rule_rep_lo=arr(t.rule_rep_lo, t.n_rules, np.int32), rule_rep_hi=arr(t.rule_rep_hi, t.n_rules, np.int32),
            cedge_iter=arr(t.cedge_iter, t.n_class_edges, np.uint8), redge_iter=arr(t.redge_iter, t.n_ref_edges, np.uint8),
            n_records=t.n_records)

    def record_of(self, state: int, count: int = 0) -> int:
        """The cache record of (state, count of finished iterations); the state itself outside counted repetitions."""
        out = C.c_int32()
        _check(lib().xg_grammar_record_of(self.h, int(state), int(count), C.byref(out)))
        return out.value

    def rule_hashes(self) -> np.ndarray:
        s = GrammarStats()
        _check(lib().xg_grammar_stats(self.h, C.byref(s)))
        out = np.zeros(s.n_rules, dtype=np.uint64)
        _check(lib().xg_grammar_get_rule_hashes(self.h, out.ctypes.data))
        return out

    def state_classes(self, depth: int = -1) -> np.ndarray:
        s = GrammarStats()
        _check(lib().xg_grammar_stats(self.h, C.byref(s)))
        out = np.zeros(s.n_states, dtype=np.int32)
        _check(lib().xg_grammar_get_state_classes(self.h, int(depth), out.ctypes.data))
        return out

    def cache_entry(self, state: int) -> dict:
        v = CacheEntryView()
        _check(lib().xg_grammar_get_cache_entry(self.h, int(state), C.byref(v)))
        out = dict(state=v.state, kind=v.kind, n_accepted=v.n_accepted, n_rejected=v.n_rejected, n_uncertain=v.n_uncertain)
        out["list"] = np.ctypeslib.as_array(C.cast(v.list, C.POINTER(C.c_int32)), shape=(v.n_list,)).copy() if v.list and v.n_list else np.zeros(0, np.int32)
        out["bitset"] = np.ctypeslib.as_array(C.cast(v.bitset, C.POINTER(C.c_uint32)), shape=(self.tokenizer.words,)).copy() if v.bitset else None
        out["uncertain"] = np.ctypeslib.as_array(C.cast(v.uncertain, C.POINTER(C.c_int32)), shape=(v.n_uncertain,)).copy() if v.n_uncertain else np.zeros(0, np.int32)
        return out

    def stats(self) -> dict:
        s = GrammarStats()
        _check(lib().xg_grammar_stats(self.h, C.byref(s)))
        d = {n: getattr(s, n) for n, _ in GrammarStats._fields_ if n not in ("kind_count", "pad")}
        d["kind_count"] = list(s.kind_count)
        return d


def jit_service(grammars: Sequence["Grammar"], stream: int = 0, wait: bool = False) -> dict:
    """Advance the just-in-time cache builds of `grammars` (see xg_jit_service)."""
    arr = (C.c_void_p * len(grammars))(*[g.h for g in grammars])
    st = JitStats()
    _check(lib().xg_jit_service(arr, len(grammars), stream, 1 if wait else 0, C.byref(st)))
    return {n: getattr(st, n) for n, _ in JitStats._fields_}


class Matcher:
    def __init__(self, grammar: Grammar, max_sets: int = 0, max_items: int = 0, stream: int = 0):
        opt = MatcherOptions(C.sizeof(MatcherOptions), max_sets, max_items)
        h = C.c_void_p()
        _check(lib().xg_matcher_create(grammar.h, C.byref(opt), stream, C.byref(h)))
        self.h = h
        self.grammar = grammar

    def reset(self, stream: int = 0):
        _check(lib().xg_matcher_reset(self.h, stream))

    def next_fill_work(self, stream: int = 0) -> dict:
        w = FillWork()
        _check(lib().xg_matcher_next_fill_work(self.h, stream, C.byref(w)))
        return {n: getattr(w, n) for n, _ in FillWork._fields_ if n != "pad"}

    def is_terminated(self, stream: int = 0) -> bool:
        out = C.c_int32(0)
        _check(lib().xg_matcher_is_terminated(self.h, stream, C.byref(out)))
        return bool(out.value)

    def close(self):
        if getattr(self, "h", None):
            lib().xg_matcher_destroy(self.h)
            self.h = None


class Batch:
    """A fixed list of matchers, marshalled once into the handle array the per-step calls take."""

    def __init__(self, matchers: Sequence[Matcher]):
        self.matchers = list(matchers)
        self.n = len(self.matchers)
        self.handles = (C.c_void_p * self.n)(*[m.h for m in self.matchers])

    def fill_next_token_bitmask(self, bitmask_ptr: int, row_stride_words: int, status_ptr: int = 0, stream: int = 0):
        _check(lib().xg_fill_next_token_bitmask(self.handles, self.n, bitmask_ptr, row_stride_words, status_ptr or None, stream))

    def fill_next_token_bitmask_static(self, bitmask_ptr: int, row_stride_words: int, status_ptr: int = 0, stream: int = 0):
        """Same masks as fill_next_token_bitmask, without any device allocation (at most
        XG_STATIC_FILL_MAX_BATCH requests; calls must not overlap on the GPU)."""
        _check(lib().xg_fill_next_token_bitmask_static(self.handles, self.n, bitmask_ptr, row_stride_words, status_ptr or None, stream))

    def fill_and_apply_token_bitmask(self, bitmask_ptr: int, row_stride_words: int, status_ptr: int, logits_ptr: int, dtype,
                                     logits_row_stride: int, stream: int = 0):
        _check(lib().xg_fill_and_apply_token_bitmask(self.handles, self.n, bitmask_ptr, row_stride_words, status_ptr or None, logits_ptr,
                                                     DTYPE_BY_NAME.get(dtype, dtype), logits_row_stride, stream))

    def accept_token(self, token_ids_ptr: int, status_ptr: int = 0, stream: int = 0, restart_on_eos: bool = False):
        if restart_on_eos:
            _check(lib().xg_accept_token_ex(self.handles, self.n, token_ids_ptr, status_ptr or None, 1, stream))
        else:
            _check(lib().xg_accept_token(self.handles, self.n, token_ids_ptr, status_ptr or None, stream))

    def accept_token_and_fill_next_bitmask(self, token_ids_ptr: int, accept_status_ptr: int, restart_on_eos: bool, bitmask_ptr: int,
                                           row_stride_words: int, fill_status_ptr: int = 0, stream: int = 0):
        _check(lib().xg_accept_token_and_fill_next_bitmask(self.handles, self.n, token_ids_ptr, accept_status_ptr or None, 1 if restart_on_eos else 0,
                                                           bitmask_ptr, row_stride_words, fill_status_ptr or None, stream))


def apply_token_bitmask(logits_ptr: int, dtype, batch: int, vocab_size: int, logits_row_stride: int, bitmask_ptr: int,
                        mask_row_stride_words: int, row_indices_ptr: int = 0, n_rows: int = 0, stream: int = 0):
    _check(lib().xg_apply_token_bitmask(logits_ptr, DTYPE_BY_NAME.get(dtype, dtype), batch, vocab_size, logits_row_stride,
                                        bitmask_ptr, mask_row_stride_words, row_indices_ptr or None, n_rows, stream))
