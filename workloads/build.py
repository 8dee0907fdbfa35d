"""Assemble the five seeded synthetic workloads: grammar text, vocabulary,
per-row token streams (prefix + decode steps) and logits.

The workloads stand in for the paper's Geoquery/FunQL, JSON-Schema and
JSON-grammar tasks and for its four models' tokenizers (Section 5.1), which
are not available here.  Only data is produced; nothing is parsed or masked.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Tuple

import numpy as np

from . import grammars as G
from .rng import SplitMix64, numpy_generator, stream

MAX_TOKEN_LEN = 16


@dataclass
class Workload:
    config: int
    name: str
    ebnf: str
    start: str
    vocab: List[bytes]  # vocab[eos] == b""
    eos: int
    batch: int
    steps: int
    prefix: np.ndarray  # [P, B] int32, -1 = nothing for that row at that position
    tokens: np.ndarray  # [steps, B] int32
    reset_before: np.ndarray  # [steps, B] bool: row restarts on a fresh document before this step
    prefix_bytes: List[bytes]  # bytes of each row's prefix
    meta: Dict[str, object] = field(default_factory=dict)

    @property
    def V(self) -> int:
        return len(self.vocab)

    def vocab_blob(self) -> Tuple[np.ndarray, np.ndarray]:
        """Concatenated token bytes (uint8) and V+1 offsets (uint64)."""
        offs = np.zeros(len(self.vocab) + 1, dtype=np.uint64)
        offs[1:] = np.cumsum([len(t) for t in self.vocab], dtype=np.uint64)
        blob = np.frombuffer(b"".join(self.vocab), dtype=np.uint8).copy()
        if blob.size == 0:
            blob = np.zeros(1, dtype=np.uint8)
        return blob, offs

    def logits_f32(self, step: int) -> np.ndarray:
        """[B, V] float32 logits ~ N(0, 4) for one step (seeded by config and step)."""
        g = numpy_generator(self.config, "logits/%d" % step)
        return (g.standard_normal((self.batch, self.V), dtype=np.float32) * 2.0).astype(np.float32)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16 bit patterns (uint16); NaN stays NaN."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    nan = (u & 0x7FFFFFFF) > 0x7F800000
    r = ((u >> 16) & 1) + 0x7FFF
    out = ((u + r) >> 16).astype(np.uint16)
    out[nan] = ((u[nan] >> 16) | 0x0040).astype(np.uint16)
    return out


# ------------------------------------------------------------------ vocabulary


def _token_len(rng: SplitMix64, lo: int, hi: int, mean: float) -> int:
    return max(lo, min(hi, 1 + rng.geometric(mean - 1.0)))


def _random_word(rng: SplitMix64, n: int) -> bytes:
    """A 'word' of at most n bytes: letters, some 2- and 3-byte code points, optional leading space."""
    out = bytearray()
    if rng.chance(0.4):
        out += b" "
    while True:
        r = rng.below(100)
        if r < 88:
            ch = bytes([rng.pick(b"abcdefghijklmnopqrstuvwxyzABCDEFGHIJKLMNOPQRSTUVWXYZ")])
        elif r < 96:
            ch = chr(rng.between(0xA0, 0x7FF)).encode()
        else:
            cp = rng.between(0x800, 0xFFFF)
            if 0xD800 <= cp <= 0xDFFF:
                cp = 0x3042
            ch = chr(cp).encode()
        if len(out) + len(ch) > n:
            break
        out += ch
    return bytes(out)


def make_vocab(
    rng: SplitMix64, V: int, corpus: bytes, lo: int = 1, hi: int = MAX_TOKEN_LEN, mean: float = 4.0,
    frac_corpus: float = 0.6, printable_random: bool = False,
) -> Tuple[List[bytes], int]:
    """256 single bytes, then V-257 distinct multi-byte tokens, then EOS (empty bytes) as id V-1."""
    assert V >= 258
    vocab: List[bytes] = [bytes([b]) for b in range(256)]
    seen = set(vocab)
    seen.add(b"")
    tries = 0
    while len(vocab) < V - 1:
        tries += 1
        n = _token_len(rng, max(lo, 2), hi, mean)
        if tries > 50 * V:  # the space of short strings is used up: lengthen
            n = min(hi, n + 2)
        if rng.chance(frac_corpus):
            o = rng.below(max(1, len(corpus) - n))
            t = corpus[o : o + n]
        elif printable_random:
            t = bytes(rng.between(0x20, 0x7E) for _ in range(n))
        else:
            t = _random_word(rng, n)
        if len(t) < 2 or len(t) > hi or t in seen:
            continue
        seen.add(t)
        vocab.append(t)
    vocab.append(b"")
    return vocab, V - 1


class Tokenizer:
    """Greedy longest-match over the vocabulary (every single byte is a token)."""

    def __init__(self, vocab: List[bytes]):
        self.table: Dict[bytes, int] = {}
        for i, t in enumerate(vocab):
            if t and t not in self.table:
                self.table[t] = i
        self.maxlen = max(len(t) for t in vocab)

    def encode(self, data: bytes) -> List[int]:
        out: List[int] = []
        i, n, tab = 0, len(data), self.table
        while i < n:
            for L in range(min(self.maxlen, n - i), 0, -1):
                t = tab.get(data[i : i + L])
                if t is not None:
                    out.append(t)
                    i += L
                    break
        return out


# ------------------------------------------------------------------ token streams


def make_streams(
    rng: SplitMix64, tok: Tokenizer, eos: int, batch: int, steps: int,
    doc_gen: Callable[[SplitMix64], bytes],
    prefix_cut: Callable[[SplitMix64, bytes, List[int]], int],
):
    """Per row: a document, cut after `prefix_cut` tokens; the rest (then EOS, then fresh
    documents from their start) supplies `steps` decode tokens."""
    prefixes: List[List[int]] = []
    tokens = np.full((steps, batch), -1, dtype=np.int32)
    reset = np.zeros((steps, batch), dtype=bool)
    for b in range(batch):
        doc = doc_gen(rng)
        ids = tok.encode(doc)
        p = max(0, min(prefix_cut(rng, doc, ids), len(ids)))
        prefixes.append(ids[:p])
        queue = ids[p:] + [eos]
        s = 0
        qi = 0
        fresh = False
        while s < steps:
            if qi == len(queue):
                queue = tok.encode(doc_gen(rng)) + [eos]
                qi = 0
                fresh = True
            tokens[s, b] = queue[qi]
            if fresh:
                reset[s, b] = True
                fresh = False
            qi += 1
            s += 1
    P = max((len(p) for p in prefixes), default=0)
    prefix = np.full((P, batch), -1, dtype=np.int32)
    for b, p in enumerate(prefixes):
        prefix[: len(p), b] = p
    return prefix, tokens, reset


# ------------------------------------------------------------------ the five configs

FULL = {
    1: dict(V=512, batch=1, steps=32),
    2: dict(V=32000, batch=8, steps=256),
    3: dict(V=128256, batch=64, steps=512),
    4: dict(V=152064, batch=128, steps=256),
    5: dict(V=128256, batch=256, steps=32),
}

NAMES = {
    1: "arith-512",
    2: "json-32k",
    3: "jsonschema-128k",
    4: "sql-152k",
    5: "ambiguous-longctx-128k",
}


def build(config: int, V: Optional[int] = None, batch: Optional[int] = None, steps: Optional[int] = None,
          prefix_scale: float = 1.0) -> Workload:
    """Build config 1..5; V / batch / steps override the full sizes (same recipe, smaller case).
    prefix_scale shrinks the prefix lengths of config 5 for small test cases."""
    full = FULL[config]
    V = V or full["V"]
    batch = batch or full["batch"]
    steps = steps or full["steps"]
    r_doc = stream(config, "documents")
    r_voc = stream(config, "vocab")
    r_corpus = stream(config, "corpus")
    meta: Dict[str, object] = {}

    def cut_tokens_upto_bytes(limit_fn):
        def cut(rng: SplitMix64, doc: bytes, ids: List[int]) -> int:
            limit = limit_fn(rng, doc)
            n = 0
            k = 0
            # ids are consumed in order; stop before exceeding `limit` bytes
            for k, t in enumerate(ids):
                n += len(vocab[t])
                if n > limit:
                    return k
            return len(ids)

        return cut

    if config == 1:
        ebnf, start = G.ARITH_EBNF, "expr"
        corpus = b" ".join(G.gen_arith_doc(r_corpus) for _ in range(40))
        vocab, eos = make_vocab(r_voc, V, corpus, lo=2, hi=6, mean=3.0, frac_corpus=0.5, printable_random=True)
        doc_gen = G.gen_arith_doc
        cut = cut_tokens_upto_bytes(lambda rng, doc: rng.between(0, 64))
    elif config == 2:
        ebnf, start = G.JSON_EBNF, "json"
        corpus = b"\n".join(G.gen_json_doc(r_corpus) for _ in range(200))
        vocab, eos = make_vocab(r_voc, V, corpus)
        doc_gen = G.gen_json_doc
        cut = cut_tokens_upto_bytes(lambda rng, doc: int(len(doc) * 0.25 * rng.unit()))
    elif config == 3:
        schema = G.gen_schema(stream(config, "schema"))
        ebnf, start = G.schema_to_ebnf(schema), "root"
        corpus = b"\n".join(G.gen_schema_instance(r_corpus, schema) for _ in range(400))
        vocab, eos = make_vocab(r_voc, V, corpus)
        doc_gen = lambda rng: G.gen_schema_instance(rng, schema)
        cut = cut_tokens_upto_bytes(lambda rng, doc: int(len(doc) * rng.unit()))
        meta["schema_fields"] = len(schema)
    elif config == 4:
        tabs, cols = G.gen_sql_names(stream(config, "names"))
        ebnf, start = G.sql_ebnf(tabs, cols), "query"
        corpus = b"\n".join(G.gen_sql_doc(r_corpus, tabs, cols) for _ in range(1500))
        vocab, eos = make_vocab(r_voc, V, corpus)
        doc_gen = lambda rng: G.gen_sql_doc(rng, tabs, cols)
        cut = cut_tokens_upto_bytes(lambda rng, doc: int(len(doc) * rng.unit()))
    elif config == 5:
        ebnf, start = G.stress_ebnf(), "json"
        corpus = b"\n".join(G.gen_stress_doc(r_corpus, 3000)[0] for _ in range(100))
        vocab, eos = make_vocab(r_voc, V, corpus)
        lo, hi = int(2048 * prefix_scale), int(8192 * prefix_scale)
        spans_of: Dict[bytes, List[Tuple[int, int]]] = {}

        def doc_gen(rng: SplitMix64) -> bytes:
            d, spans = G.gen_stress_doc(rng, hi + 600)
            spans_of[d] = spans
            return d

        def limit_fn(rng: SplitMix64, doc: bytes) -> int:
            target = rng.between(lo, hi)
            spans = [s for s in spans_of.get(doc, []) if lo <= s[0] and s[1] <= hi and s[1] - s[0] > 2]
            if spans and rng.chance(0.25):  # end inside an ambiguous segment
                s = rng.pick(spans)
                target = rng.between(s[0] + 1, s[1] - 1)
            return target

        cut = cut_tokens_upto_bytes(limit_fn)
    else:
        raise ValueError("config must be 1..5")

    tok = Tokenizer(vocab)
    prefix, tokens, reset = make_streams(r_doc, tok, eos, batch, steps, doc_gen, cut)
    prefix_bytes = [b"".join(vocab[t] for t in prefix[:, b] if t >= 0) for b in range(batch)]
    return Workload(
        config=config, name=NAMES[config], ebnf=ebnf, start=start, vocab=vocab, eos=eos, batch=batch,
        steps=steps, prefix=prefix, tokens=tokens, reset_before=reset, prefix_bytes=prefix_bytes, meta=meta,
    )
