"""Pins for the CPU oracle: the paper's worked examples, brute-force enumeration on tiny
grammars, closed forms and invariants.  None of these re-uses the oracle's own formulas:
the expected values come from the paper's text (tests/golden), from a bottom-up language
enumerator written here, from hand-built automata, or from Python's json module."""
import itertools
import json
import os

import numpy as np
import pytest

import oracle
import workloads
from workloads.rng import SplitMix64

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def load_golden(name):
    g = {"grammar": [], "sets": {}, "next": {}, "other": {}}
    for line in open(os.path.join(GOLDEN, name), encoding="utf-8"):
        line = line.rstrip("\n")
        if not line or line.startswith("#"):
            continue
        if line.startswith("grammar: "):
            g["grammar"].append(line[len("grammar: "):])
        elif line.startswith("next "):
            k, v = line[5:].split(":", 1)
            g["next"][int(k)] = v.split()
        elif "|" in line and line.split("|")[0].strip().isdigit():
            k, item = line.split("|", 1)
            g["sets"].setdefault(int(k), []).append(item.strip())
        else:
            k, v = line.split(":", 1)
            g["other"][k.strip()] = v.strip()
    return g


def single_byte_vocab():
    return oracle.Vocab([bytes([b]) for b in range(256)] + [b""], eos=256)


def valid_bytes(seq, vocab):
    m = oracle.bits(seq.mask(vocab), 257)
    return {bytes([b]) for b in range(256) if m[b]}, bool(m[256])


# ---------------------------------------------------------------- the paper's worked examples


def test_section1_example_chart_and_pruning():
    gold = load_golden("section1_example.txt")
    g = oracle.Grammar("\n".join(gold["grammar"]), gold["other"]["start"])
    s = oracle.Sequence_(g)
    text = gold["other"]["input"].encode()
    assert s.advance(text[:1])
    set1 = set(s.set_items(1))
    # exactly the four states the paper lists, plus the augmented start item
    assert set1 - {"$ -> A . ; 0"} == set(gold["sets"][1])
    assert len(gold["sets"][1]) == 4
    assert s.advance(text[1:])
    for item in gold["sets"][2]:
        assert item in s.set_items(2)
    # pruning: the completed item is gone; after "a" and after "aa" the pruned charts coincide
    p = oracle.Sequence_(g, pruned=True)
    assert p.advance(b"a")
    k1 = p.key()
    assert gold["other"]["pruned-away-after-set-1"] not in k1
    assert p.set_items(p.num_sets - 1) == sorted(["A -> A . B ; 0", "B -> . a ; 1"])
    assert p.set_items(0) == sorted(["$ -> . A ; 0", "A -> . A B ; 0"])
    keys = [k1]
    for _ in range(5):
        assert p.advance(b"a")
        keys.append(p.key())
    assert len(set(keys)) == 1 and p.num_sets == 2
    vocab = oracle.Vocab([b"a", b"b", b"aa", b"ab", b""], eos=4)
    for seq in (s, p):
        assert list(oracle.bits(seq.mask(vocab), 5)) == [True, False, True, False, True]


def test_section32_example_chart():
    gold = load_golden("section32_example.txt")
    g = oracle.Grammar("\n".join(gold["grammar"]), gold["other"]["start"])
    s = oracle.Sequence_(g)
    assert not s.accepting
    assert s.advance(b"a") and not s.accepting
    assert s.advance(b"b") and s.accepting
    for k, items in gold["sets"].items():
        for item in items:
            assert item in s.set_items(k), (k, item)
    assert "B -> . b ; 1" in s.set_items(1) and "B -> b . ; 1" in s.set_items(2)
    assert not s.advance(b"b")  # nothing may follow
    assert s.num_sets == 3  # a rejected advance leaves the chart as it was


def test_figure1_example_next_bytes():
    gold = load_golden("figure1_example.txt")
    g = oracle.Grammar("\n".join(gold["grammar"]), gold["other"]["start"])
    vocab = single_byte_vocab()
    text = gold["other"]["input"].encode()
    for pruned in (False, True):
        s = oracle.Sequence_(g, pruned=pruned)
        for pos in range(len(text) + 1):
            ok, acc = valid_bytes(s, vocab)
            assert ok == {x.encode() for x in gold["next"][pos]}, pos
            assert acc == (pos == int(gold["other"]["accepting-after"]))
            if pos < len(text):
                assert s.advance(text[pos:pos + 1])


def test_section33_example_mask_after_open_brace():
    gold = load_golden("section33_example.txt")
    g = oracle.Grammar("\n".join(gold["grammar"]), gold["other"]["start"])
    vocab = single_byte_vocab()
    for pruned in (False, True):
        s = oracle.Sequence_(g, pruned=pruned)
        assert s.advance(gold["other"]["input"].encode())
        ok, acc = valid_bytes(s, vocab)
        assert ok == {x.encode() for x in gold["other"]["valid-single-bytes"].split()}
        assert not acc


# ---------------------------------------------------------------- brute force on tiny grammars


def enumerate_language(rules, start, max_len):
    """All sentences of length <= max_len, by a bottom-up fixpoint on sets of strings
    (terminals are the one-character strings that are not keys of `rules`)."""
    lang = {x: set() for x in rules}
    changed = True
    while changed:
        changed = False
        for x, alts in rules.items():
            for alt in alts:
                partial = {""}
                for sym in alt:
                    opts = lang[sym] if sym in rules else {sym}
                    partial = {p + o for p in partial for o in opts if len(p) + len(o) <= max_len}
                    if not partial:
                        break
                new = partial - lang[x]
                if new:
                    lang[x] |= new
                    changed = True
    return lang[start]


def to_ebnf(rules):
    lines = []
    for x, alts in rules.items():
        parts = []
        for alt in alts:
            parts.append(" ".join(s if s in rules else '"%s"' % s for s in alt) if alt else '""')
        lines.append("%s ::= %s" % (x, " | ".join(parts)))
    return "\n".join(lines)


TINY = {
    "finite": ({"S": [["a", "b"], ["a", "T", "c"], ["T"]], "T": [["b", "b"], ["c"], []]}, "abc", 4, 8),
    "anbn": ({"S": [["a", "S", "b"], []]}, "ab", 5, 16),
    "dyck": ({"S": [["S", "(", "S", ")"], []]}, "()", 5, 16),
    "palindrome": ({"P": [["a", "P", "a"], ["b", "P", "b"], ["a"], ["b"], []]}, "ab", 5, 16),
    "ambiguous": ({"E": [["E", "E"], ["E", "+", "E"], ["(", "E", ")"], ["a"]]}, "a+()", 2, 9, 2),
    "nullable": ({"S": [["A", "B", "A"], ["S", "c"]], "A": [["a"], []], "B": [["b", "B"], ["A", "A"]]}, "abc", 4, 9),
    "leftrec": ({"L": [["L", ",", "x"], ["x"]]}, "x,", 5, 12),
    "useless": ({"S": [["a", "S"], ["b"], ["U", "a"]], "U": [["U", "b"]], "X": [["a"]]}, "ab", 4, 10),
}


@pytest.mark.parametrize("name", sorted(TINY))
def test_brute_force_viable_prefixes(name):
    rules, alphabet, max_prefix, L = TINY[name][:4]
    max_tok = TINY[name][4] if len(TINY[name]) > 4 else 3  # L covers the longest completion needed
    start = next(iter(rules))
    lang = enumerate_language(rules, start, L)
    prefixes_of_lang = {s[:i] for s in lang for i in range(len(s) + 1)}
    g = oracle.Grammar(to_ebnf(rules), start)
    tokens = ["".join(t) for n in range(1, max_tok + 1) for t in itertools.product(alphabet, repeat=n)]
    vocab = oracle.Vocab([t.encode() for t in tokens] + [b""], eos=len(tokens))
    checked = 0
    for n in range(max_prefix + 1):
        for tup in itertools.product(alphabet, repeat=n):
            w = "".join(tup)
            for pruned in (False, True):
                s = oracle.Sequence_(g, pruned=pruned)
                ok = s.advance(w.encode()) if w else True
                assert ok == (w in prefixes_of_lang), (w, pruned)
                if not ok:
                    continue
                m = oracle.bits(s.mask(vocab), len(tokens) + 1)
                for i, t in enumerate(tokens):
                    # every viable string of this length has a completion within L (L is chosen so)
                    assert bool(m[i]) == ((w + t) in prefixes_of_lang), (w, t, pruned)
                assert bool(m[len(tokens)]) == (w in lang), (w, pruned)
                assert s.accepting == (w in lang)
                checked += 1
    assert checked > 10


# ---------------------------------------------------------------- closed forms


def test_dyck_closed_form():
    g = oracle.Grammar('S ::= S "(" S ")" | ""', "S")
    vocab = oracle.Vocab([b"(", b")", b"()", b")(", b"))", b"(((", b"())", b""], eos=7)
    rng = SplitMix64(7)
    for pruned in (False, True):
        s = oracle.Sequence_(g, pruned=pruned)
        depth = 0
        for step in range(300):
            m = list(oracle.bits(s.mask(vocab), 8))
            expect = [True, depth > 0, True, depth > 0, depth > 1, True, depth > 0, depth == 0]
            assert m == expect, (step, depth)
            if depth > 0 and rng.chance(0.5):
                assert s.advance(b")")
                depth -= 1
            else:
                assert s.advance(b"(")
                depth += 1
        if pruned:
            assert s.num_sets <= depth + 2  # one surviving set per open bracket


def test_decimal_numbers_against_hand_dfa():
    ebnf = 'num ::= "-"? ( "0" | [1-9] [0-9]* ) ( "." [0-9]+ )? ( [eE] [+\\-]? [0-9]+ )?'
    g = oracle.Grammar(ebnf, "num")
    # states: 0 start, 1 after '-', 2 after '0', 3 in int digits, 4 after '.', 5 in frac, 6 after e,
    # 7 after e sign, 8 in exp digits
    def step(q, c):
        d = c.isdigit()
        if q == 0:
            return 1 if c == "-" else 2 if c == "0" else 3 if d else None
        if q == 1:
            return 2 if c == "0" else 3 if d else None
        if q in (2, 3):
            if q == 3 and d:
                return 3
            return 4 if c == "." else 6 if c in "eE" else None
        if q == 4:
            return 5 if d else None
        if q == 5:
            return 5 if d else 6 if c in "eE" else None
        if q == 6:
            return 7 if c in "+-" else 8 if d else None
        if q == 7:
            return 8 if d else None
        if q == 8:
            return 8 if d else None
    accepting = {2, 3, 5, 8}
    alphabet = "0123456789-+.eE"
    tokens = [a for a in alphabet] + [a + b for a in "01-.e+" for b in "05.eE-"]
    vocab = oracle.Vocab([t.encode() for t in tokens] + [b""], eos=len(tokens))
    rng = SplitMix64(11)
    for trial in range(60):
        s = oracle.Sequence_(g, pruned=bool(trial & 1))
        q = 0
        for _ in range(12):
            m = oracle.bits(s.mask(vocab), len(tokens) + 1)
            for i, t in enumerate(tokens):
                qq = q
                for c in t:
                    qq = step(qq, c) if qq is not None else None
                assert bool(m[i]) == (qq is not None), (trial, t, q)  # every DFA state is live
            assert bool(m[len(tokens)]) == (q in accepting)
            options = [c for c in alphabet if step(q, c) is not None]
            if not options:
                break
            c = rng.pick(options)
            assert s.advance(c.encode())
            q = step(q, c)


def test_arithmetic_against_hand_automaton():
    g = oracle.Grammar(workloads.grammars.ARITH_EBNF, "expr")
    vocab = single_byte_vocab()
    rng = SplitMix64(3)
    for trial in range(20):
        s = oracle.Sequence_(g, pruned=bool(trial & 1))
        depth, want_operand, in_number = 0, True, False
        for _ in range(80):
            ok, acc = valid_bytes(s, vocab)
            expect = set()
            if want_operand:
                expect |= {b"("} | {bytes([d]) for d in b"0123456789"}
            else:
                expect |= {b"+", b"-", b"*", b"/"}
                if in_number:
                    expect |= {bytes([d]) for d in b"0123456789"}
                if depth > 0:
                    expect |= {b")"}
            assert ok == expect
            assert acc == (not want_operand and depth == 0)
            c = rng.pick(sorted(expect))
            assert s.advance(c)
            if c == b"(":
                depth += 1
                in_number = False
            elif c == b")":
                depth -= 1
                in_number = False
            elif c in b"+-*/":
                want_operand, in_number = True, False
            else:
                want_operand, in_number = False, True


# ---------------------------------------------------------------- invariants on the workloads


def _walk(config, rows, n_steps, check_every, **kw):
    w = workloads.build(config, **kw)
    g = oracle.Grammar(w.ebnf, w.start)
    vocab = oracle.Vocab(w.vocab, w.eos)
    lens = np.array([len(t) for t in w.vocab])
    order = np.argsort(lens, kind="stable")
    index = {t: i for i, t in enumerate(w.vocab)}
    for b in range(min(rows, w.batch)):
        full, pruned = oracle.Sequence_(g), oracle.Sequence_(g, pruned=True)
        assert full.advance(w.prefix_bytes[b]) and pruned.advance(w.prefix_bytes[b])
        for i in range(min(n_steps, w.steps)):
            t = int(w.tokens[i, b])
            if w.reset_before[i, b]:
                full, pruned = oracle.Sequence_(g), oracle.Sequence_(g, pruned=True)
            if i % check_every == 0:
                m = full.mask(vocab)
                # I1: pruning does not change the mask (Section 4.1, "preserving ... completeness")
                assert np.array_equal(m, pruned.mask(vocab)), (config, b, i)
                bits = oracle.bits(m, w.V)
                # I4: the token the document continues with is valid
                assert bits[t], (config, b, i, w.vocab[t])
                # I3: viable prefixes are prefix-closed
                for tok in np.nonzero(bits)[0][:: max(1, int(bits.sum()) // 200)]:
                    bt = w.vocab[tok]
                    for k in range(1, len(bt)):
                        j = index.get(bt[:k])
                        if j is not None:
                            assert bits[j], (bt, bt[:k])
                # a live, non-accepting state has at least one valid single byte
                assert bits[:256].any() or full.accepting
            if t == w.eos:
                assert full.accepting and pruned.accepting
                continue
            assert full.advance(w.vocab[t]) and pruned.advance(w.vocab[t])
        yield w, full, pruned


def test_invariants_config1():
    for w, full, pruned in _walk(1, rows=1, n_steps=32, check_every=1):
        assert pruned.total_items <= full.total_items


def test_invariants_config2():
    for w, full, pruned in _walk(2, rows=3, n_steps=96, check_every=8, V=6000, batch=3, steps=96):
        assert pruned.total_items < full.total_items / 10  # the chart no longer grows with the prefix


def test_invariants_config3():
    for w, full, pruned in _walk(3, rows=2, n_steps=120, check_every=12, V=6000, batch=2, steps=120):
        assert pruned.total_items < full.total_items / 5


def test_invariants_config4():
    for w, full, pruned in _walk(4, rows=2, n_steps=100, check_every=10, V=6000, batch=2, steps=100):
        assert pruned.total_items < full.total_items


def test_invariants_config5():
    for w, full, pruned in _walk(5, rows=2, n_steps=24, check_every=4, V=5000, batch=2, steps=24, prefix_scale=0.25):
        assert pruned.total_items < full.total_items / 5


def test_hrr_grammar_keeps_pruned_chart_constant():
    # rules of the forms A -> c, A -> B a, A -> empty (Section 4.1) leave nothing to keep
    g = oracle.Grammar('A ::= B "a" | "c"\nB ::= A "b" | ""', "A")
    p, f = oracle.Sequence_(g, pruned=True), oracle.Sequence_(g)
    sizes = set()
    text = b"c" + b"ba" * 200
    for i in range(len(text)):
        assert p.advance(text[i:i + 1]) and f.advance(text[i:i + 1])
        if i > 2:
            sizes.add((p.num_sets, p.total_items, i % 2))
    assert len(sizes) == 2 and p.total_items <= 4
    assert f.num_sets == len(text) + 1 and f.total_items > 400


def test_sampling_valid_tokens_keeps_prefix_completable():
    # I2 (Section 6: "100% structural compliance"): after any masked-valid token the mask is never
    # all-zero, and greedy use of the shortest valid token reaches an accepting state.
    w = workloads.build(2, V=3000, batch=1, steps=8)
    g = oracle.Grammar(w.ebnf, w.start)
    vocab = oracle.Vocab(w.vocab, w.eos)
    rng = SplitMix64(99)
    s = oracle.Sequence_(g, pruned=True)
    for step in range(150):
        bits = oracle.bits(s.mask(vocab), w.V)
        assert bits.any(), step
        choices = np.nonzero(bits)[0]
        t = int(choices[rng.below(len(choices))])
        if t == w.eos:
            break
        assert s.advance(w.vocab[t])
    # close everything: prefer closers, then the shortest valid token
    for step in range(400):
        if s.accepting:
            break
        bits = oracle.bits(s.mask(vocab), w.V)
        assert bits.any()
        pick = None
        for c in (b'"', b"}", b"]", b"0", b":", b"e"):
            if s.check(c):
                n = s.clone()
                n.advance(c)
                pick = c
                break
        if pick is None:
            pick = w.vocab[int(np.nonzero(bits[:256])[0][0])]
        assert s.advance(pick)
    assert s.accepting


def test_grammar_form_invariance():
    # I5: one language written several ways gives one mask
    forms = [
        'list ::= "[" ( item ( "," item )* )? "]"\nitem ::= [a-c]+ | list',
        'list ::= "[" "]" | "[" items "]"\nitems ::= items "," item | item\nitem ::= word | list\nword ::= word [a-c] | [a-c]',
        'list ::= "[" opt "]"\nopt ::= "" | item rest\nrest ::= "" | "," item rest\nitem ::= [a-c] tail | list\n'
        'tail ::= "" | [a-c] tail\nunused ::= "z" unused\ndead ::= dead "q"',
    ]
    gs = [oracle.Grammar(f, "list") for f in forms]
    toks = [bytes(t) for n in (1, 2) for t in itertools.product(b"[],abz", repeat=n)]
    vocab = oracle.Vocab(toks + [b""], eos=len(toks))
    rng = SplitMix64(5)
    for trial in range(30):
        seqs = [oracle.Sequence_(g, pruned=bool(i & 1)) for i, g in enumerate(gs)]
        for _ in range(14):
            masks = [s.mask(vocab) for s in seqs]
            assert all(np.array_equal(masks[0], m) for m in masks[1:])
            bits = oracle.bits(masks[0], len(toks))
            choices = np.nonzero(bits)[0]
            if len(choices) == 0:
                break
            t = toks[int(choices[rng.below(len(choices))])]
            assert all(s.advance(t) for s in seqs)


def test_json_acceptance_agrees_with_json_module():
    g = oracle.Grammar(workloads.grammars.JSON_EBNF, "json")
    rng = SplitMix64(2024)
    agree_reject = 0
    for trial in range(40):
        doc = workloads.grammars.gen_json_value(rng, 0, 4)
        s = oracle.Sequence_(g, pruned=bool(trial & 1))
        assert s.advance(doc) and s.accepting, doc
        json.loads(doc.decode("utf-8"))
        for _ in range(12):
            pos = rng.below(len(doc))
            bad = bytearray(doc)
            bad[pos] = rng.below(256)
            bad = bytes(bad)
            try:
                json.loads(bad.decode("utf-8"))
                py_ok = True
            except (ValueError, UnicodeDecodeError):
                py_ok = False
            s2 = oracle.Sequence_(g)
            ours = s2.advance(bad) and s2.accepting
            assert ours == py_ok, bad
            agree_reject += (not py_ok)
    assert agree_reject > 100


# ---------------------------------------------------------------- error paths and mask application


def test_grammar_errors():
    with pytest.raises(oracle.OracleGrammarError) as e:
        oracle.Grammar('a ::= "x" b', "a")
    assert e.value.code == oracle.UNDEFINED_SYMBOL
    with pytest.raises(oracle.OracleGrammarError) as e:
        oracle.Grammar('a ::= "x" a', "a")
    assert e.value.code == oracle.EMPTY_LANGUAGE
    with pytest.raises(oracle.OracleGrammarError) as e:
        oracle.Grammar('a ::= "x', "a")
    assert e.value.code == oracle.SYNTAX
    with pytest.raises(oracle.OracleGrammarError) as e:
        oracle.Grammar('a ::= "x"', "nope")
    assert e.value.code == oracle.UNDEFINED_SYMBOL


def test_empty_and_duplicate_tokens():
    g = oracle.Grammar('s ::= "ab" | "a"', "s")
    vocab = oracle.Vocab([b"a", b"", b"a", b"ab", b"", b"b"], eos=4)
    s = oracle.Sequence_(g)
    assert list(oracle.bits(s.mask(vocab), 6)) == [True, False, True, True, False, False]
    s.advance(b"a")
    assert list(oracle.bits(s.mask(vocab), 6)) == [False, False, False, False, True, True]


def test_apply_mask_against_numpy_where():
    rng = np.random.default_rng(5)
    B, V = 3, 77
    words = (V + 31) // 32
    mask = rng.integers(0, 2**32, size=(B, words), dtype=np.uint64).astype(np.uint32)
    bits = np.stack([oracle.bits(mask[b], V) for b in range(B)])
    f = rng.standard_normal((B, V)).astype(np.float32)
    f[0, 3], f[1, 5], f[2, 7], f[0, 9] = np.nan, np.inf, -np.inf, -0.0
    out = oracle.apply_mask(mask, f, "fp32")
    expect = np.where(bits, f, np.float32(-np.inf))
    assert np.array_equal(out.view(np.uint32), expect.view(np.uint32))
    h = workloads.f32_to_bf16_bits(f)
    h[1, 11] = 0x7FC1  # a NaN with a payload
    out = oracle.apply_mask(mask, h, "bf16")
    expect = np.where(bits, h, np.uint16(0xFF80))
    assert np.array_equal(out, expect)
    # -inf really is 0xFF80 in bfloat16 and 0xFF800000 in float32
    assert np.array([0xFF800000], dtype=np.uint32).view(np.float32)[0] == -np.inf
    assert (np.array([0xFF80], dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)[0] == -np.inf
