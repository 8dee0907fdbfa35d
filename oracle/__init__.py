"""TEST INFRASTRUCTURE — Python wrapper of the CPU oracle (earley_oracle.cpp).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library never does and shares no code with it.

The oracle follows the paper's definitions: Earley sets with predict / scan / complete
(Section 3.2), the logits mask over the whole vocabulary (Sections 3.3 and 4.1), the
useless-rule removal of Section 4.5, and - in `pruned=True` sequences - the Compact step
of Section 4.2.3 in the reading of Figure 3's caption.
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

OK, BAD_ARG, SYNTAX, UNDEFINED_SYMBOL, EMPTY_LANGUAGE = 0, 1, 2, 3, 4


class OracleGrammarError(Exception):
    def __init__(self, code: int, msg: str):
        super().__init__("%d: %s" % (code, msg))
        self.code = code


def build(force: bool = False) -> str:
    """Compile the oracle's shared library next to its source (g++ -O2, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fopenmp", "-shared", "-fPIC", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, sz = C.c_void_p, C.c_size_t
        L.orc_grammar_new.argtypes = [C.c_char_p, sz, C.c_char_p, C.POINTER(vp), C.c_char_p, sz]
        L.orc_grammar_new.restype = C.c_int
        L.orc_grammar_free.argtypes = [vp]
        for f in ("orc_grammar_num_rules", "orc_grammar_num_nonterminals", "orc_grammar_num_dotted"):
            getattr(L, f).argtypes = [vp]
            getattr(L, f).restype = C.c_int
        L.orc_grammar_rule_text.argtypes = [vp, C.c_int, C.c_char_p, sz]
        L.orc_grammar_rule_text.restype = sz
        L.orc_vocab_new.argtypes = [vp, vp, C.c_uint32, C.c_int32]
        L.orc_vocab_new.restype = vp
        L.orc_vocab_free.argtypes = [vp]
        L.orc_seq_new.argtypes = [vp, C.c_int]
        L.orc_seq_new.restype = vp
        L.orc_seq_clone.argtypes = [vp]
        L.orc_seq_clone.restype = vp
        L.orc_seq_free.argtypes = [vp]
        L.orc_seq_advance.argtypes = [vp, C.c_char_p, sz]
        L.orc_seq_advance.restype = C.c_int
        L.orc_seq_accepting.argtypes = [vp]
        L.orc_seq_accepting.restype = C.c_int
        for f in ("orc_seq_num_sets", "orc_seq_total_items", "orc_seq_peak_items"):
            getattr(L, f).argtypes = [vp]
            getattr(L, f).restype = sz
        L.orc_seq_set_size.argtypes = [vp, sz]
        L.orc_seq_set_size.restype = sz
        L.orc_seq_set_text.argtypes = [vp, sz, C.c_char_p, sz]
        L.orc_seq_set_text.restype = sz
        L.orc_seq_key_text.argtypes = [vp, C.c_char_p, sz]
        L.orc_seq_key_text.restype = sz
        L.orc_seq_check_bytes.argtypes = [vp, C.c_char_p, sz]
        L.orc_seq_check_bytes.restype = C.c_int
        L.orc_seq_mask.argtypes = [vp, vp, vp, C.c_int]
        L.orc_max_threads.restype = C.c_int
        L.orc_apply_mask.argtypes = [vp, sz, vp, C.c_int, C.c_uint32, C.c_uint32, sz]
        _lib = L
    return _lib


def max_threads() -> int:
    return lib().orc_max_threads()


class Grammar:
    """A reduced grammar (Section 4.5) parsed from the grammar text."""

    def __init__(self, ebnf: str, start: str):
        src = ebnf.encode("latin-1") if isinstance(ebnf, str) else ebnf
        out = C.c_void_p()
        err = C.create_string_buffer(512)
        rc = lib().orc_grammar_new(src, len(src), start.encode(), C.byref(out), err, 512)
        if rc != OK:
            raise OracleGrammarError(rc, err.value.decode(errors="replace"))
        self._h = out

    def __del__(self):
        if getattr(self, "_h", None):
            lib().orc_grammar_free(self._h)
            self._h = None

    @property
    def num_rules(self) -> int:
        return lib().orc_grammar_num_rules(self._h)

    @property
    def num_nonterminals(self) -> int:
        return lib().orc_grammar_num_nonterminals(self._h)

    @property
    def num_dotted(self) -> int:
        return lib().orc_grammar_num_dotted(self._h)

    def rules(self) -> List[str]:
        out = []
        for r in range(self.num_rules):
            n = lib().orc_grammar_rule_text(self._h, r, None, 0)
            buf = C.create_string_buffer(n + 1)
            lib().orc_grammar_rule_text(self._h, r, buf, n + 1)
            out.append(buf.value.decode("latin-1"))
        return out


class Vocab:
    def __init__(self, tokens: Sequence[bytes], eos: int = -1):
        self.tokens = list(tokens)
        self.eos = eos
        offs = np.zeros(len(tokens) + 1, dtype=np.uint64)
        offs[1:] = np.cumsum([len(t) for t in tokens], dtype=np.uint64)
        blob = np.frombuffer(b"".join(tokens) + b"\0", dtype=np.uint8).copy()
        self._h = C.c_void_p(lib().orc_vocab_new(blob.ctypes.data, offs.ctypes.data, len(tokens), eos))

    def __del__(self):
        if getattr(self, "_h", None):
            lib().orc_vocab_free(self._h)
            self._h = None

    def __len__(self):
        return len(self.tokens)


class Sequence_:
    """One decoding sequence: the Earley chart of the bytes advanced so far."""

    def __init__(self, grammar: Grammar, pruned: bool = False, _h=None):
        self.grammar = grammar
        self.pruned = pruned
        self._h = _h if _h is not None else C.c_void_p(lib().orc_seq_new(grammar._h, 1 if pruned else 0))

    def __del__(self):
        if getattr(self, "_h", None):
            lib().orc_seq_free(self._h)
            self._h = None

    def clone(self) -> "Sequence_":
        return Sequence_(self.grammar, self.pruned, C.c_void_p(lib().orc_seq_clone(self._h)))

    def advance(self, data: bytes) -> bool:
        """Append bytes; False (and no change) if the result is not a viable prefix."""
        return bool(lib().orc_seq_advance(self._h, data, len(data)))

    def check(self, data: bytes) -> bool:
        """Would these (non-empty) bytes keep the prefix viable?  No change to the sequence."""
        return bool(lib().orc_seq_check_bytes(self._h, data, len(data)))

    @property
    def accepting(self) -> bool:
        return bool(lib().orc_seq_accepting(self._h))

    @property
    def num_sets(self) -> int:
        return lib().orc_seq_num_sets(self._h)

    @property
    def total_items(self) -> int:
        return lib().orc_seq_total_items(self._h)

    @property
    def peak_items(self) -> int:
        return lib().orc_seq_peak_items(self._h)

    def set_items(self, k: int) -> List[str]:
        n = lib().orc_seq_set_text(self._h, k, None, 0)
        buf = C.create_string_buffer(n + 1)
        lib().orc_seq_set_text(self._h, k, buf, n + 1)
        return [l for l in buf.value.decode("latin-1").split("\n") if l]

    def key(self) -> str:
        n = lib().orc_seq_key_text(self._h, None, 0)
        buf = C.create_string_buffer(n + 1)
        lib().orc_seq_key_text(self._h, buf, n + 1)
        return buf.value.decode("latin-1")

    def mask(self, vocab: Vocab, threads: int = 0) -> np.ndarray:
        """uint32 words, bit t&31 of word t>>5 set iff token t is valid (pad bits 0)."""
        out = np.zeros((len(vocab) + 31) // 32, dtype=np.uint32)
        lib().orc_seq_mask(self._h, vocab._h, out.ctypes.data, threads)
        return out


def apply_mask(mask: np.ndarray, logits: np.ndarray, dtype: str) -> np.ndarray:
    """Return a copy of `logits` ([B, V], uint16 bf16 bit patterns or float32) with the
    entries of invalid tokens replaced by -inf; mask is [B, words] uint32."""
    assert mask.dtype == np.uint32 and mask.ndim == 2
    out = np.ascontiguousarray(logits).copy()
    B, V = out.shape
    code = {"bf16": 0, "fp32": 1}[dtype]
    assert (code == 0 and out.dtype == np.uint16) or (code == 1 and out.dtype == np.float32)
    m = np.ascontiguousarray(mask)
    lib().orc_apply_mask(m.ctypes.data, m.shape[1], out.ctypes.data, code, B, V, V)
    return out


def bits(mask_words: np.ndarray, V: int) -> np.ndarray:
    """Unpack mask words into a bool array of length V."""
    b = np.unpackbits(mask_words.view(np.uint8), bitorder="little")
    return b[:V].astype(bool)
