"""Thin ctypes binding of the C-ABI in include/fmt.h: argument marshalling only.

Every step of the path runs in the CUDA library; PyTorch is used by callers for device memory
and streams (tensors are passed here as raw device pointers).  There is no CPU fallback: if the
library cannot be loaded, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np

from ._build import LIB, build

FMT_OK = 0
ERR_INVALID_ARG, ERR_GRAMMAR_SYNTAX, ERR_UNDEFINED_SYMBOL, ERR_EMPTY_LANGUAGE = 1, 2, 3, 4
ERR_OOM, ERR_CUDA, ERR_CAPACITY, ERR_TOKEN_REJECTED, ERR_FINISHED = 5, 6, 7, 8, 9
BF16, FP32 = 0, 1

EXPORTS = [
    "fmt_compile", "fmt_json_schema_to_ebnf", "fmt_compile_json_schema", "fmt_grammar_destroy", "fmt_grammar_get_info", "fmt_grammar_copy_table", "fmt_grammar_automaton_match",
    "fmt_state_create", "fmt_state_destroy", "fmt_state_reset", "fmt_state_advance", "fmt_state_forced_bytes", "fmt_fill_mask",
    "fmt_apply_mask", "fmt_fill_and_apply", "fmt_state_cache_clear", "fmt_state_ci_cache_clear", "fmt_state_set_wait_limit", "fmt_state_copy_counters", "fmt_state_query", "fmt_state_copy_chart", "fmt_get_stats",
    "fmt_state_set_profiling", "fmt_state_read_profile", "fmt_state_read_profile_series", "fmt_fill_mask_noalloc", "fmt_last_error",
]


class FmtError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__("fmt error %d: %s" % (code, msg))
        self.code = code


class CompileOptions(C.Structure):
    _fields_ = [("host_only", C.c_uint32), ("no_dfa_terminals", C.c_uint32), ("reserved", C.c_uint32 * 6)]


class StateOptions(C.Structure):
    _fields_ = [
        ("cache_disable", C.c_uint32), ("max_states", C.c_uint32), ("max_mask_rows", C.c_uint32),
        ("chart_words", C.c_uint32), ("pool_words", C.c_uint64), ("sweep_states", C.c_uint32),
        ("roots_enable", C.c_uint32), ("max_roots", C.c_uint32), ("root_max_items", C.c_uint32),
        ("root_max_origins", C.c_uint32), ("wait_limit_log2", C.c_uint32), ("cache_keep_when_full", C.c_uint32),
    ]


class GrammarInfo(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in (
        "n_nonterminals", "n_rules", "n_dotted", "n_classes", "n_nullable", "vocab_size", "mask_words",
        "trie_nodes", "trie_depth", "n_byte_classes", "n_empty_tokens", "start_nullable", "n_automata", "n_automaton_states")]


class Stats(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in (
        "steps_advanced", "fills", "fills_computed", "fills_from_cache", "fills_shared", "states_cached",
        "mask_rows_cached", "pool_words_used", "chart_items_max", "chart_sets_max", "capacity_errors",
        "big_mode_units", "sweep_transitions", "sweep_states", "advances_cached", "roots", "root_sweeps",
        "rows_mask_only", "rows_from_root", "rows_plain", "walk_transitions", "walk_states", "walk_frames",
        "fills_aborted", "device_bytes", "earley_step_cycles", "advance_chart_words")] + [("diag", C.c_uint64 * 16), ("cache_flushes", C.c_uint64)]

    def as_dict(self):
        d = {n: int(getattr(self, n)) for n, _ in self._fields_ if n != "diag"}
        d["diag"] = [int(x) for x in self.diag]
        return d


class Profile(C.Structure):
    _fields_ = [("advance_ms", C.c_double), ("sweep_ms", C.c_double), ("apply_ms", C.c_double),
                ("advance_launches", C.c_uint64), ("sweep_launches", C.c_uint64), ("apply_launches", C.c_uint64),
                ("roots_ms", C.c_double), ("roots_launches", C.c_uint64)]


_lib = None


def lib():
    """Load (building first if needed) the shared library; raises if that is impossible."""
    global _lib
    if _lib is None:
        path = build()
        L = C.CDLL(path)
        vp, sz, u32, i32 = C.c_void_p, C.c_size_t, C.c_uint32, C.c_int32
        L.fmt_compile.argtypes = [C.c_char_p, sz, C.c_char_p, vp, vp, u32, i32, C.POINTER(CompileOptions), C.POINTER(vp)]
        L.fmt_grammar_destroy.argtypes = [vp]
        L.fmt_grammar_destroy.restype = None
        L.fmt_grammar_get_info.argtypes = [vp, C.POINTER(GrammarInfo)]
        L.fmt_grammar_copy_table.argtypes = [vp, C.c_int, vp, sz, C.POINTER(sz)]
        L.fmt_grammar_automaton_match.argtypes = [vp, u32, C.c_char_p, sz, C.POINTER(C.c_int), C.c_char_p, sz]
        L.fmt_state_create.argtypes = [vp, u32, C.POINTER(StateOptions), vp, C.POINTER(vp)]
        L.fmt_state_destroy.argtypes = [vp]
        L.fmt_state_destroy.restype = None
        L.fmt_state_reset.argtypes = [vp, vp, u32, vp]
        L.fmt_state_advance.argtypes = [vp, vp, vp, vp]
        L.fmt_state_forced_bytes.argtypes = [vp, vp, sz, vp, u32, vp]
        L.fmt_fill_mask.argtypes = [vp, vp, sz, vp]
        L.fmt_apply_mask.argtypes = [vp, sz, vp, C.c_int, u32, u32, sz, vp]
        L.fmt_fill_and_apply.argtypes = [vp, vp, sz, vp, C.c_int, sz, vp]
        L.fmt_state_cache_clear.argtypes = [vp, vp]
        L.fmt_state_ci_cache_clear.argtypes = [vp, vp]
        L.fmt_state_set_wait_limit.argtypes = [vp, u32]
        L.fmt_state_copy_counters.argtypes = [vp, C.c_int, vp, sz, C.POINTER(sz), vp]
        L.fmt_state_query.argtypes = [vp, vp, vp, vp, vp, vp, vp]
        L.fmt_state_copy_chart.argtypes = [vp, u32, vp, sz, C.POINTER(sz), vp]
        L.fmt_get_stats.argtypes = [vp, C.POINTER(Stats), vp]
        L.fmt_state_set_profiling.argtypes = [vp, C.c_int]
        L.fmt_state_read_profile.argtypes = [vp, C.POINTER(Profile)]
        L.fmt_state_read_profile_series.argtypes = [vp, C.c_int, vp, sz, C.POINTER(sz)]
        L.fmt_fill_mask_noalloc.argtypes = [vp, vp, vp, u32, vp, vp, vp]
        L.fmt_last_error.restype = C.c_char_p
        for name in EXPORTS:
            if name not in ("fmt_grammar_destroy", "fmt_state_destroy", "fmt_last_error"):
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def _check(rc: int):
    if rc != FMT_OK:
        raise FmtError(rc, lib().fmt_last_error().decode(errors="replace"))


def _ptr(x) -> Optional[int]:
    """Device pointer of a torch tensor, or a raw integer / None."""
    if x is None:
        return None
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    return int(x)


_TABLE_DTYPES = {0: np.uint32, 1: np.uint8, 2: np.uint32, 3: np.uint32, 4: np.uint32, 5: np.uint32, 6: np.uint8,
                 7: np.uint32, 8: np.uint16, 9: np.uint32, 10: np.uint8, 11: np.uint16, 12: np.uint8, 13: np.uint32}


def json_schema_to_ebnf(schema) -> str:
    """fmt_json_schema_to_ebnf: grammar text (start rule "root") for the instances of a JSON schema."""
    src = schema.encode("utf-8") if isinstance(schema, str) else bytes(schema)
    n = C.c_size_t()
    _check(lib().fmt_json_schema_to_ebnf(src, len(src), None, 0, C.byref(n)))
    buf = C.create_string_buffer(max(n.value, 1))
    _check(lib().fmt_json_schema_to_ebnf(src, len(src), buf, n.value, C.byref(n)))
    return buf.raw[: n.value].decode("latin-1")


class Grammar:
    """fmt_compile: grammar text + vocabulary -> device tables and byte trie."""

    @classmethod
    def from_json_schema(cls, schema, vocab: Sequence[bytes], eos: int = -1, host_only: bool = False, dfa: bool = True) -> "Grammar":
        """fmt_compile_json_schema: the instances of a JSON schema as the grammar."""
        self = cls.__new__(cls)
        src = schema.encode("utf-8") if isinstance(schema, str) else bytes(schema)
        offs = np.zeros(len(vocab) + 1, dtype=np.uint64)
        offs[1:] = np.cumsum([len(t) for t in vocab], dtype=np.uint64)
        blob = np.frombuffer(b"".join(vocab) + b"\0", dtype=np.uint8).copy()
        opt = CompileOptions()
        opt.host_only = 1 if host_only else 0
        opt.no_dfa_terminals = 0 if dfa else 1
        h = C.c_void_p()
        _check(lib().fmt_compile_json_schema(src, len(src), blob.ctypes.data, offs.ctypes.data, len(vocab), eos,
                                             C.byref(opt), C.byref(h)))
        self._h = h
        self.V = len(vocab)
        self.eos = eos
        self.mask_words = (self.V + 31) // 32
        return self

    def __init__(self, ebnf, start: str, vocab: Sequence[bytes], eos: int = -1, host_only: bool = False, dfa: bool = True):
        src = ebnf.encode("latin-1") if isinstance(ebnf, str) else bytes(ebnf)
        offs = np.zeros(len(vocab) + 1, dtype=np.uint64)
        offs[1:] = np.cumsum([len(t) for t in vocab], dtype=np.uint64)
        blob = np.frombuffer(b"".join(vocab) + b"\0", dtype=np.uint8).copy()
        opt = CompileOptions()
        opt.host_only = 1 if host_only else 0
        opt.no_dfa_terminals = 0 if dfa else 1
        h = C.c_void_p()
        _check(lib().fmt_compile(src, len(src), start.encode(), blob.ctypes.data, offs.ctypes.data, len(vocab), eos,
                                 C.byref(opt), C.byref(h)))
        self._h = h
        self.V = len(vocab)
        self.eos = eos
        self.mask_words = (self.V + 31) // 32

    def close(self):
        if getattr(self, "_h", None):
            lib().fmt_grammar_destroy(self._h)
            self._h = None

    __del__ = close

    def info(self) -> GrammarInfo:
        out = GrammarInfo()
        _check(lib().fmt_grammar_get_info(self._h, C.byref(out)))
        return out

    def automaton_name(self, k: int) -> str:
        name = C.create_string_buffer(256)
        acc = C.c_int()
        _check(lib().fmt_grammar_automaton_match(self._h, k, b"", 0, C.byref(acc), name, 256))
        return name.value.decode("latin-1")

    def automaton_accepts(self, k: int, data: bytes) -> bool:
        """fmt_grammar_automaton_match: is `data` a sentence of the regular non-terminal automaton k stands for?"""
        acc = C.c_int()
        _check(lib().fmt_grammar_automaton_match(self._h, k, bytes(data), len(data), C.byref(acc), None, 0))
        return bool(acc.value)

    def table(self, which: int) -> np.ndarray:
        n = C.c_size_t()
        _check(lib().fmt_grammar_copy_table(self._h, which, None, 0, C.byref(n)))
        buf = np.zeros(max(n.value, 1), dtype=np.uint8)
        _check(lib().fmt_grammar_copy_table(self._h, which, buf.ctypes.data, n.value, C.byref(n)))
        return buf[: n.value].view(_TABLE_DTYPES[which])


class State:
    """fmt_state_*: a batch of sequences on the device."""

    def __init__(self, grammar: Grammar, batch: int, stream=None, cache: bool = True, max_states: int = 0,
                 max_mask_rows: int = 0, pool_words: int = 0, chart_words: int = 0, sweep_states: int = 0,
                 roots: bool = False, max_roots: int = 0, root_max_items: int = 0, root_max_origins: int = 0,
                 wait_limit_log2: int = 0, keep_when_full: bool = False):
        self.grammar = grammar
        self.batch = batch
        opt = StateOptions()
        opt.cache_disable = 0 if cache else 1
        opt.max_states = max_states
        opt.max_mask_rows = max_mask_rows
        opt.pool_words = pool_words
        opt.chart_words = chart_words
        opt.sweep_states = sweep_states
        opt.roots_enable = 1 if roots else 0
        opt.max_roots = max_roots
        opt.root_max_items = root_max_items
        opt.root_max_origins = root_max_origins
        opt.wait_limit_log2 = wait_limit_log2
        opt.cache_keep_when_full = 1 if keep_when_full else 0
        h = C.c_void_p()
        _check(lib().fmt_state_create(grammar._h, batch, C.byref(opt), _ptr(stream), C.byref(h)))
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            lib().fmt_state_destroy(self._h)
            self._h = None

    __del__ = close

    def reset(self, rows_dev=None, n: Optional[int] = None, stream=None):
        """rows_dev: device int32/uint32 tensor of row indices, or None for rows 0..n-1 (default all)."""
        if rows_dev is None:
            n = self.batch if n is None else n
        elif n is None:
            n = rows_dev.numel()
        _check(lib().fmt_state_reset(self._h, _ptr(rows_dev), n, _ptr(stream)))

    def advance(self, token_ids_dev, status_dev=None, stream=None):
        _check(lib().fmt_state_advance(self._h, _ptr(token_ids_dev), _ptr(status_dev), _ptr(stream)))

    def forced_bytes(self, bytes_dev, len_dev, max_len: int = 32, stride_bytes: Optional[int] = None, stream=None):
        """fmt_state_forced_bytes: per row the bytes every continuation must begin with (uint8 [batch, stride], uint32 [batch])."""
        stride = stride_bytes if stride_bytes is not None else int(bytes_dev.shape[-1])
        _check(lib().fmt_state_forced_bytes(self._h, _ptr(bytes_dev), stride, _ptr(len_dev), max_len, _ptr(stream)))

    def fill_mask(self, mask_dev, stride_words: Optional[int] = None, stream=None):
        stride = self.grammar.mask_words if stride_words is None else stride_words
        _check(lib().fmt_fill_mask(self._h, _ptr(mask_dev), stride, _ptr(stream)))

    def fill_and_apply(self, logits_dev, dtype: int, row_stride: Optional[int] = None, mask_dev=None,
                       stride_words: Optional[int] = None, stream=None):
        stride = self.grammar.mask_words if stride_words is None else stride_words
        rs = self.grammar.V if row_stride is None else row_stride
        _check(lib().fmt_fill_and_apply(self._h, _ptr(mask_dev), stride, _ptr(logits_dev), dtype, rs, _ptr(stream)))

    def cache_clear(self, stream=None):
        _check(lib().fmt_state_cache_clear(self._h, _ptr(stream)))

    def ci_cache_clear(self, stream=None):
        _check(lib().fmt_state_ci_cache_clear(self._h, _ptr(stream)))

    def counters(self, which: int = 0, stream=None) -> np.ndarray:
        """fmt_state_copy_counters: the raw device counters (0: the state's, 1: its root sweeps')."""
        n = C.c_size_t()
        _check(lib().fmt_state_copy_counters(self._h, which, None, 0, C.byref(n), _ptr(stream)))
        buf = np.zeros(n.value, dtype=np.uint32)
        _check(lib().fmt_state_copy_counters(self._h, which, buf.ctypes.data, n.value, C.byref(n), _ptr(stream)))
        return buf

    def set_wait_limit(self, log2_polls: int):
        _check(lib().fmt_state_set_wait_limit(self._h, log2_polls))

    def query(self, stream=None):
        B = self.batch
        acc = np.zeros(B, np.uint8)
        fin = np.zeros(B, np.uint8)
        ns = np.zeros(B, np.uint32)
        ni = np.zeros(B, np.uint32)
        sid = np.zeros(B, np.int32)
        _check(lib().fmt_state_query(self._h, acc.ctypes.data, fin.ctypes.data, ns.ctypes.data, ni.ctypes.data,
                                     sid.ctypes.data, _ptr(stream)))
        return {"accepting": acc, "finished": fin, "n_sets": ns, "n_items": ni, "state_id": sid}

    def chart(self, row: int, stream=None) -> dict:
        """The row's pruned chart: {'sets': [[(dotted_rule, origin), ...], ...], 'accepting': bool}."""
        n = C.c_size_t()
        _check(lib().fmt_state_copy_chart(self._h, row, None, 0, C.byref(n), _ptr(stream)))
        buf = np.zeros(n.value, dtype=np.uint32)
        _check(lib().fmt_state_copy_chart(self._h, row, buf.ctypes.data, n.value, C.byref(n), _ptr(stream)))
        m = int(buf[0])
        off = buf[8 : 8 + m + 1]
        items = buf[8 + m + 1 :]
        sets = [[(int(x & 0xFFFF), int(x >> 16)) for x in items[off[k] : off[k + 1]]] for k in range(m)]
        return {"sets": sets, "accepting": bool(buf[2] & 1), "words": int(buf[5])}

    def chart_words(self, row: int, stream=None) -> np.ndarray:
        """The raw words of the row's pruned chart (the layout fmt_state_copy_chart documents)."""
        n = C.c_size_t()
        _check(lib().fmt_state_copy_chart(self._h, row, None, 0, C.byref(n), _ptr(stream)))
        buf = np.zeros(n.value, dtype=np.uint32)
        _check(lib().fmt_state_copy_chart(self._h, row, buf.ctypes.data, n.value, C.byref(n), _ptr(stream)))
        return buf

    def set_profiling(self, on: bool, step_cycles: bool = False):
        """Kernel timing with CUDA events; `step_cycles` also counts the SM cycles inside Earley steps."""
        _check(lib().fmt_state_set_profiling(self._h, (1 if on else 0) | (2 if step_cycles else 0)))

    def read_profile_series(self, kind: int) -> np.ndarray:
        """Per-launch durations (ms) of one kind of kernel (0 advance, 1 sweep, 2 masking, 3 entries); call before read_profile."""
        n = C.c_size_t()
        _check(lib().fmt_state_read_profile_series(self._h, kind, None, 0, C.byref(n)))
        buf = np.zeros(max(n.value, 1), dtype=np.float32)
        _check(lib().fmt_state_read_profile_series(self._h, kind, buf.ctypes.data, n.value, C.byref(n)))
        return buf[: n.value]

    def read_profile(self) -> dict:
        out = Profile()
        _check(lib().fmt_state_read_profile(self._h, C.byref(out)))
        return {n: getattr(out, n) for n, _ in out._fields_}

    def stats(self, stream=None) -> dict:
        out = Stats()
        _check(lib().fmt_get_stats(self._h, C.byref(out), _ptr(stream)))
        return out.as_dict()


def apply_mask(mask_dev, logits_dev, dtype: int, batch: int, V: int, stride_words: Optional[int] = None,
               row_stride: Optional[int] = None, stream=None):
    """fmt_apply_mask on raw device buffers."""
    stride = (V + 31) // 32 if stride_words is None else stride_words
    rs = V if row_stride is None else row_stride
    _check(lib().fmt_apply_mask(_ptr(mask_dev), stride, _ptr(logits_dev), dtype, batch, V, rs, _ptr(stream)))


NOALLOC_MAX_CHARTS = 64


def fill_mask_noalloc(grammar: Grammar, charts_dev, chart_offsets: Sequence[int], mask_dev, status_dev=None, stream=None):
    """fmt_fill_mask_noalloc: masks for charts already in device memory, using only the scratch
    array built into the library (no allocation; see include/fmt.h for who needs that and why).
    chart_offsets: n+1 word offsets into charts_dev; mask_dev: [n, ceil(V/32)] dense."""
    offs = np.ascontiguousarray(chart_offsets, dtype=np.uint64)
    n = len(offs) - 1
    _check(lib().fmt_fill_mask_noalloc(grammar._h, _ptr(charts_dev), offs.ctypes.data, n, _ptr(mask_dev),
                                       _ptr(status_dev), _ptr(stream)))
