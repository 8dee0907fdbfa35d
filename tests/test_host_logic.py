"""CPU-only checks of the library's host side: the shared object loads and exports the whole
C-ABI, and fmt_compile's grammar reduction and trie construction (host_only mode) are right."""
import os
import re

import numpy as np
import pytest

import paper_2506_01151_b200 as fmt
import workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    L = fmt.lib()
    declared = set()
    for name in os.listdir(os.path.join(ROOT, "include")):
        text = open(os.path.join(ROOT, "include", name)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        declared |= set(re.findall(r"\b(fmt_[a-z_0-9]+)\s*\(", text))
    assert declared, "no declarations found"
    for sym in sorted(declared):
        assert hasattr(L, sym), sym
    assert declared == set(fmt.EXPORTS)


def walk(child_off, node_byte, data: bytes):
    n = 0
    for c in data:
        lo, hi = child_off[n], child_off[n + 1]
        kids = node_byte[lo:hi]
        j = np.searchsorted(kids, c)
        if j >= len(kids) or kids[j] != c:
            return None
        n = lo + j
    return n


@pytest.mark.parametrize("config,kw", [(1, {}), (2, dict(V=8000, batch=2, steps=4))])
def test_trie_is_a_valid_csr_trie(config, kw):
    w = workloads.build(config, **kw)
    vocab = list(w.vocab)
    vocab[300] = vocab[299]  # a duplicate byte string
    g = fmt.Grammar(w.ebnf, w.start, vocab, w.eos, host_only=True)
    info = g.info()
    child_off, node_byte, parent = g.table(0), g.table(1), g.table(2)
    tok_off, tok_ids = g.table(3), g.table(4)
    T = info.trie_nodes
    assert len(child_off) == T + 1 and len(node_byte) == T and child_off[0] == 1 and child_off[T] == T
    assert (np.diff(child_off.astype(np.int64)) >= 0).all()
    for n in range(0, T, max(1, T // 2000)):
        kids = node_byte[child_off[n]:child_off[n + 1]]
        assert (np.diff(kids.astype(np.int32)) > 0).all()  # distinct, ascending
        for c in range(child_off[n], child_off[n + 1]):
            assert parent[c] == n
    # every non-empty token ends at exactly one node, which lists it
    assert len(tok_ids) == info.vocab_size - info.n_empty_tokens
    assert sorted(tok_ids.tolist()) == [t for t in range(len(vocab)) if vocab[t]]
    for t in list(range(0, len(vocab), 37)) + [299, 300]:
        if not vocab[t]:
            continue
        n = walk(child_off, node_byte, vocab[t])
        assert n is not None and t in tok_ids[tok_off[n]:tok_off[n + 1]]
    n = walk(child_off, node_byte, vocab[300])
    assert {299, 300} <= set(tok_ids[tok_off[n]:tok_off[n + 1]].tolist())
    assert info.trie_depth == max(len(t) for t in vocab)
    # breadth-first numbering: every depth is one contiguous range, parents come before children
    lvl = g.table(5)
    assert len(lvl) == info.trie_depth + 2 and lvl[0] == 0 and lvl[1] == 1 and lvl[-1] == T
    depth = np.zeros(T, dtype=np.int64)
    for n in range(1, T):
        assert parent[n] < n
        depth[n] = depth[parent[n]] + 1
    for L in range(info.trie_depth + 1):
        assert (depth[lvl[L]:lvl[L + 1]] == L).all() and lvl[L] < lvl[L + 1]
    # token -> node is the inverse of the per-node token lists
    tok_node = g.table(9)
    assert len(tok_node) == len(vocab)
    for t in range(0, len(vocab), 23):
        if vocab[t]:
            assert tok_node[t] == walk(child_off, node_byte, vocab[t])
        else:
            assert tok_node[t] == 0xFFFFFFFF
    # bytes in one class behave alike: for this grammar digits must share a class, '(' and ')' must not
    eq = g.table(10)
    assert info.n_byte_classes == len(set(eq.tolist()))


def test_grammar_reduction_and_nullability():
    text = '''
    s ::= a b c | s "x"
    a ::= "a" | ""
    b ::= a a | "b" b
    c ::= ( "c" | d )*
    d ::= "d"+
    dead ::= dead "q"
    unused ::= "z"
    '''
    g = fmt.Grammar(text, "s", [b"a", b""], eos=1, host_only=True, dfa=False)  # (the rules as written: no automata)
    info = g.info()
    nullable = g.table(6)
    assert info.start_nullable == 1
    # $, s, a, b, c, the star's helper, the group of the star, d, the plus's helper: dead and unused are gone
    assert info.n_nonterminals == 9
    assert info.n_nullable == nullable.sum() == 6  # $ s a b c and the star helper
    kinds = g.table(7) >> 30
    assert (kinds == 0).sum() == info.n_rules  # one completed position per rule


@pytest.mark.parametrize("text,start,vocab,eos,code", [
    ('a ::= "x" b', "a", [b"x"], -1, fmt.ERR_UNDEFINED_SYMBOL),
    ('a ::= "x" a', "a", [b"x"], -1, fmt.ERR_EMPTY_LANGUAGE),
    ('a ::= "x', "a", [b"x"], -1, fmt.ERR_GRAMMAR_SYNTAX),
    ('a ::= [z-a]', "a", [b"x"], -1, fmt.ERR_GRAMMAR_SYNTAX),
    ('a ::= ( "x"', "a", [b"x"], -1, fmt.ERR_GRAMMAR_SYNTAX),
    ('a ::= "x"', "b", [b"x"], -1, fmt.ERR_UNDEFINED_SYMBOL),
    ('a ::= "x"', "a", [b"x", b"y"], 1, fmt.ERR_INVALID_ARG),  # EOS must have no bytes
    ('a ::= "x"', "a", [b"x" * 33], -1, fmt.ERR_CAPACITY),
    ('a ::= "x"', "a", [b"x"], 5, fmt.ERR_INVALID_ARG),
])
def test_compile_errors(text, start, vocab, eos, code):
    with pytest.raises(fmt.FmtError) as e:
        fmt.Grammar(text, start, vocab, eos, host_only=True)
    assert e.value.code == code, str(e.value)


def test_host_only_grammar_cannot_make_states():
    g = fmt.Grammar('a ::= "x"', "a", [b"x", b""], 1, host_only=True)
    with pytest.raises(fmt.FmtError) as e:
        fmt.State(g, 1)
    assert e.value.code == fmt.ERR_INVALID_ARG


def test_all_five_workload_grammars_compile_like_the_oracle_accepts_them():
    """The compiler puts bytes that no terminal of the grammar tells apart into one class and keeps
    one transition per class.  Checked against the oracle: at several points of a sentence, two
    bytes of the same class are either both accepted as the next byte or both refused, and the
    classes are not vacuous (bytes the oracle treats differently sit in different classes)."""
    import oracle

    for c in range(1, 6):
        w = workloads.build(c, V=2000, batch=1, steps=2, prefix_scale=0.05)
        g = fmt.Grammar(w.ebnf, w.start, w.vocab, w.eos, host_only=True)
        og = oracle.Grammar(w.ebnf, w.start)
        info = g.info()
        assert info.vocab_size == w.V and info.n_empty_tokens == 1
        assert info.n_dotted > 0 and og.num_rules > 0
        cls = g.table(10)
        assert len(cls) == 256 and int(cls.max()) + 1 == info.n_byte_classes
        text = bytes(w.prefix_bytes[0])
        split = 0
        for cut in sorted({0, 1, len(text) // 3, len(text) // 2, len(text)}):
            seq = oracle.Sequence_(og)
            assert seq.advance(text[:cut])
            ok = np.array([seq.check(bytes([b])) for b in range(256)])
            for k in range(info.n_byte_classes):
                members = ok[cls == k]
                assert members.all() or not members.any(), (c, cut, k)
            split += len({(int(cls[b]), bool(ok[b])) for b in range(256)}) > 1
        assert split > 0, c
