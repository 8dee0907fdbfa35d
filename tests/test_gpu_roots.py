"""GPU tests of what sits between the chart and the mask: the context-independent mask cache
(Section 4.3), the canonical form of pruned charts (Section 5.2: different token sequences, same
state), the device's Compact on the paper's Section 1 example, and the give-up path of the fill's
bounded waits.  Expected masks come from the CPU oracle."""
import numpy as np
import pytest

import oracle
import workloads

pytestmark = pytest.mark.gpu


def _torch():
    import torch

    return torch, torch.device("cuda:0")


def _mask_of(st, g, batch):
    torch, dev = _torch()
    m = torch.zeros((batch, g.mask_words), dtype=torch.int32, device=dev)
    st.fill_mask(m)
    return m.cpu().numpy().view(np.uint32)


def _advance(st, tokens):
    torch, dev = _torch()
    status = torch.full((len(tokens),), -7, dtype=torch.int32, device=dev)
    st.advance(torch.tensor(tokens, dtype=torch.int32, device=dev), status)
    return status.cpu().numpy().tolist()


def _feed_bytes(st, seqs, rows_text):
    """Advance row b by the bytes rows_text[b], one single-byte token (ids 0..255) per call."""
    n = max(len(t) for t in rows_text)
    for k in range(n):
        ids = [t[k] if k < len(t) else -1 for t in rows_text]
        got = _advance(st, ids)
        assert all(x == 0 for x in got), (k, got)
    for b, t in enumerate(rows_text):
        if t:
            assert seqs[b].advance(bytes(t))


def test_rows_with_different_charts_share_the_context_independent_part():
    """Two JSON prefixes that end inside a string under different nestings have different charts
    but the same last Earley set up to the names of its origins: the second row must find the
    first row's entry (no second vocabulary sweep, almost no Earley steps) and both masks must
    equal the oracle's."""
    import paper_2506_01151_b200 as fmt

    w = workloads.build(2, V=6000, batch=2, steps=4)
    g = fmt.Grammar(w.ebnf, w.start, w.vocab, w.eos)
    og, ov = oracle.Grammar(w.ebnf, w.start), oracle.Vocab(w.vocab, w.eos)
    st = fmt.State(g, 2, cache=False, roots=True)  # no state cache: every fill computes both rows
    seqs = [oracle.Sequence_(og) for _ in range(2)]
    _feed_bytes(st, seqs, [list(b'{"a": "x'), []])
    got = _mask_of(st, g, 2)
    for b in range(2):
        assert np.array_equal(got[b], seqs[b].mask(ov)), b
    s0 = st.stats()
    assert s0["roots"] >= 2 and s0["root_sweeps"] >= 2 and s0["sweep_transitions"] > 0
    # row 1 now reaches the inside of a string by another way
    _feed_bytes(st, seqs, [[], list(b'[[1, {"k": ["yz')])
    q = st.query()
    assert st.chart_words(0).tolist() != st.chart_words(1).tolist()
    got = _mask_of(st, g, 2)
    for b in range(2):
        assert np.array_equal(got[b], seqs[b].mask(ov)), b
    s1 = st.stats()
    # the only sweeps since are of sets the first row's walk met on its way (entered then, swept now)
    assert s1["root_sweeps"] - s0["root_sweeps"] <= s0["roots"] - s0["root_sweeps"]
    assert s1["rows_from_root"] - s0["rows_from_root"] == 2 and s1["rows_plain"] == s0["rows_plain"]
    # what is left per row is the closing quote and what may follow it in that row's context
    assert s1["walk_transitions"] - s0["walk_transitions"] < 1000
    assert s1["capacity_errors"] == 0 and s1["fills_aborted"] == 0
    # the same with the cache for context-independent masks switched off: same masks, by the long way
    st2 = fmt.State(g, 2, cache=False, roots=False)
    seqs2 = [oracle.Sequence_(og) for _ in range(2)]
    _feed_bytes(st2, seqs2, [list(b'{"a": "x'), list(b'[[1, {"k": ["yz')])
    assert np.array_equal(_mask_of(st2, g, 2), got)
    s2 = st2.stats()
    assert s2["roots"] == 0 and s2["rows_plain"] == 2 and s2["walk_transitions"] > s1["walk_transitions"] - s0["walk_transitions"]


@pytest.mark.parametrize("config", [1, 2])
def test_chart_is_the_same_under_any_token_segmentation(config):
    """Section 5.2: different token sequences that spell the same bytes must reach the same pruned
    state.  Rows 0..B-1 take the workload's greedy tokens, rows B..2B-1 the same bytes one byte
    token at a time: after every token the two charts must be equal word for word and share one
    cache id."""
    import paper_2506_01151_b200 as fmt

    w = workloads.build(config, V=4000, batch=3, steps=40) if config == 2 else workloads.build(1)
    B = w.batch
    g = fmt.Grammar(w.ebnf, w.start, w.vocab, w.eos)
    st = fmt.State(g, 2 * B)

    def both(tokens):
        ids = [int(t) for t in tokens]
        assert _advance(st, ids + [-1] * B) == [0] * (2 * B)
        texts = [w.vocab[t] if t >= 0 and t != w.eos else b"" for t in ids]
        for k in range(max(len(t) for t in texts) if texts else 0):
            assert _advance(st, [-1] * B + [t[k] if k < len(t) else -1 for t in texts]) == [0] * (2 * B)

    checked = 0
    for p in range(w.prefix.shape[0]):
        both(w.prefix[p])
    for i in range(w.steps):
        if w.reset_before[i].any() or (w.tokens[i] == w.eos).any():
            break
        both(w.tokens[i])
        q = st.query()
        for b in range(B):
            a, c = st.chart_words(b), st.chart_words(B + b)
            assert a.tolist() == c.tolist(), (i, b)
            assert q["state_id"][b] == q["state_id"][B + b] >= 0, (i, b)
            checked += 1
    assert checked >= 8 * B


def _item_texts(g, sets):
    """Items of a device chart as the oracle prints them, for a grammar whose rules are told apart
    by their shapes: "LHS -> rhs with . ; origin"."""
    info, lhs = g.table(7), g.table(8)
    D = len(info)
    kind = lambda d: int(info[d]) >> 30
    arg = lambda d: int(info[d]) & 0xFFFF
    starts = [d for d in range(D) if d == 0 or kind(d - 1) == 0]
    rules = []  # (lhs id, [symbols]) with symbols ("t", class) or ("n", id)
    for s in starts:
        syms, d = [], s
        while kind(d) != 0:
            syms.append(("t", arg(d)) if kind(d) == 1 else ("n", arg(d)))
            d += 1
        rules.append((int(lhs[s]), syms, s))
    name = {int(lhs[0]): "$"}
    for l, syms, _ in rules:
        if len(syms) == 1 and syms[0][0] == "t":
            name[l] = "B"
    for l, syms, _ in rules:
        if l not in name:
            name[l] = "A"
    out = []
    for items in sets:
        texts = []
        for d, o in items:
            l, syms, s = next(r for r in reversed(rules) if r[2] <= d)
            rhs = [name[x[1]] if x[0] == "n" else "a" for x in syms]
            rhs.insert(d - s, ".")
            texts.append("%s -> %s ; %d" % (name[l], " ".join(rhs), o))
        out.append(sorted(texts))
    return out


def test_device_compact_on_the_section1_example():
    """Section 1 of the paper: A -> A B | B, B -> a.  After "a" the pruned chart keeps, of set 0,
    the items that still wait for an A, and the last set; after "aa" set 1 is gone and the chart
    is the one after "a" again, so a, aa, ..., aaaaaa share one cache id.  Compared with the
    oracle's pruned chart item by item."""
    import paper_2506_01151_b200 as fmt

    text = 'A ::= A B | B\nB ::= "a"'
    vocab = [b"a", b"b", b"aa", b"ab", b""]
    g = fmt.Grammar(text, "A", vocab, 4, dfa=False)  # the rules as written (as a whole this language is regular: one automaton otherwise)
    og = oracle.Grammar(text, "A")
    st = fmt.State(g, 1)
    p = oracle.Sequence_(og, pruned=True)
    ids = []
    for n in range(1, 7):
        assert _advance(st, [0]) == [0]
        assert p.advance(b"a")
        ch = st.chart(0)
        got = _item_texts(g, ch["sets"])
        want = [sorted(p.set_items(k)) for k in range(p.num_sets)]
        assert got == want, (n, got, want)
        assert ch["accepting"] == p.accepting
        ids.append(int(st.query()["state_id"][0]))
    assert got[0] == sorted(["$ -> . A ; 0", "A -> . A B ; 0"]) and len(got) == 2
    assert got[1] == sorted(["A -> A . B ; 0", "B -> . a ; 1"])
    assert len(set(ids)) == 1 and ids[0] >= 0
    # and by the two-byte token
    st.reset()
    assert _advance(st, [2]) == [0]
    assert int(st.query()["state_id"][0]) == ids[0]
    got = _mask_of(st, g, 1)[0]
    assert got[0] == 0b10101  # a, aa and EOS


def test_rows_sharing_a_broken_computation_get_no_guessed_mask():
    """Two rows with the same chart share one mask computation.  When that computation runs out of
    room (a table of Earley sets far too small) neither row may get a partial mask: each mask is
    all-zero, or it equals the oracle's."""
    import paper_2506_01151_b200 as fmt

    w = workloads.build(2, V=6000, batch=2, steps=4)
    g = fmt.Grammar(w.ebnf, w.start, w.vocab, w.eos)
    og, ov = oracle.Grammar(w.ebnf, w.start), oracle.Vocab(w.vocab, w.eos)
    for roots in (False, True):
        st = fmt.State(g, 2, sweep_states=16, roots=roots)
        seqs = [oracle.Sequence_(og) for _ in range(2)]
        _feed_bytes(st, seqs, [list(b'{"a": [1, '), list(b'{"a": [1, ')])
        assert st.chart_words(0).tolist() == st.chart_words(1).tolist()
        got = _mask_of(st, g, 2)
        want = seqs[0].mask(ov)
        s = st.stats()
        assert s["fills_shared"] == 1
        for b in range(2):
            assert not got[b].any() or np.array_equal(got[b], want), (roots, b)
        if s["capacity_errors"]:
            assert not got.any(), roots
        else:
            assert np.array_equal(got[0], want) and np.array_equal(got[1], want), roots
    assert s["capacity_errors"] > 0 or s["roots"] > 0  # 16 sets are not enough for JSON unless the root carries the work


@pytest.mark.parametrize("roots", [False, True], ids=["from_chart", "ci_cache"])
def test_a_wait_that_runs_out_gives_up_cleanly(roots):
    """Every wait inside the fill's kernels is a poll with a limit.  With a limit of two polls the
    waits run out although nothing is wrong: the fill must come back, report itself aborted and
    hand out all-zero masks (never a wrong bit); with the default limits the next fill is exact."""
    import paper_2506_01151_b200 as fmt

    w = workloads.build(2, V=6000, batch=4, steps=4)
    g = fmt.Grammar(w.ebnf, w.start, w.vocab, w.eos)
    og, ov = oracle.Grammar(w.ebnf, w.start), oracle.Vocab(w.vocab, w.eos)
    st = fmt.State(g, 4, cache=False, roots=roots)
    seqs = [oracle.Sequence_(og) for _ in range(4)]
    _feed_bytes(st, seqs, [list(b'{"a": "x'), list(b"[1, 2"), list(b'{"k": tr'), list(b"[[")])
    want = np.stack([s.mask(ov) for s in seqs])
    st.set_wait_limit(1)
    aborted = 0
    for _ in range(3):
        before = st.stats()["fills_aborted"]
        got = _mask_of(st, g, 4)
        if st.stats()["fills_aborted"] > before:
            aborted += 1
            assert not got.any()
        else:
            assert np.array_equal(got, want)
    assert aborted >= 1
    st.set_wait_limit(0)
    assert np.array_equal(_mask_of(st, g, 4), want)
    assert _advance(st, [ord("y"), ord("]"), ord("u"), ord("]")]) == [0, 0, 0, 0]
    for b, c in enumerate(b"y]u]"):
        assert seqs[b].advance(bytes([c]))
    assert np.array_equal(_mask_of(st, g, 4), np.stack([s.mask(ov) for s in seqs]))
    assert st.stats()["capacity_errors"] == 0


def _oracle_forced_run(seq, limit):
    """Brute force on the oracle: while the text is not a sentence and exactly one of the 256 bytes
    can follow, take it."""
    run = []
    s = seq.clone()
    while len(run) < limit and not s.accepting:
        ok = [b for b in range(256) if s.check(bytes([b]))]
        if len(ok) != 1:
            break
        run.append(ok[0])
        assert s.advance(bytes(ok))
    return run


def test_forced_bytes_equal_the_oracles_brute_force():
    """Jump-ahead on the JSON-Schema workload (keys and punctuation are fixed by the schema): after
    every step, each row's run equals the oracle's, found byte by byte over all 256 bytes; and the
    run is the common prefix of every valid token's bytes."""
    import paper_2506_01151_b200 as fmt

    torch, dev = _torch()
    w = workloads.build(3, V=6000, batch=6, steps=48)
    g = fmt.Grammar(w.ebnf, w.start, w.vocab, w.eos)
    og, ov = oracle.Grammar(w.ebnf, w.start), oracle.Vocab(w.vocab, w.eos)
    st = fmt.State(g, w.batch)
    seqs = [oracle.Sequence_(og) for _ in range(w.batch)]
    for p in range(w.prefix.shape[0]):
        assert all(x == 0 for x in _advance(st, [int(x) for x in w.prefix[p]]))
    for b in range(w.batch):
        assert seqs[b].advance(w.prefix_bytes[b])
    out = torch.full((w.batch, 32), 0xEE, dtype=torch.uint8, device=dev)
    lens = torch.full((w.batch,), 99, dtype=torch.int32, device=dev)
    longest, nonzero = 0, 0
    for i in range(w.steps):
        r = np.nonzero(w.reset_before[i])[0]
        if len(r):
            st.reset(torch.from_numpy(r.astype(np.int32)).to(dev))
            for b in r:
                seqs[int(b)] = oracle.Sequence_(og)
        _advance(st, [int(x) for x in w.tokens[i]])
        fin = [int(w.tokens[i, b]) == w.eos for b in range(w.batch)]
        for b in range(w.batch):
            t = int(w.tokens[i, b])
            if t != w.eos and t >= 0:
                assert seqs[b].advance(w.vocab[t])
        before = [st.chart_words(b).tolist() for b in range(w.batch)]
        out.fill_(0xEE)
        st.forced_bytes(out, lens, 32)
        got_len, got = lens.cpu().numpy(), out.cpu().numpy()
        assert [st.chart_words(b).tolist() for b in range(w.batch)] == before  # the rows did not move
        for b in range(w.batch):
            if fin[b]:
                assert got_len[b] == 0
                continue
            want = _oracle_forced_run(seqs[b], 32)
            assert got[b, : got_len[b]].tolist() == want, (i, b, bytes(want))
            assert (got[b, got_len[b]:] == 0xEE).all()
            longest = max(longest, len(want))
            nonzero += len(want) > 0
            if want and i % 8 == 0:  # every valid token agrees with the run as far as both go
                m = seqs[b].mask(ov)
                for t in np.nonzero(oracle.bits(m, len(w.vocab)))[0][:200]:
                    tb = w.vocab[int(t)]
                    k = min(len(tb), len(want))
                    assert list(tb[:k]) == want[:k], (i, b, tb)
    assert longest >= 4 and nonzero >= 10  # key literals give real runs
    # a shorter limit cuts the run, it does not change it
    st.forced_bytes(out, lens, 3)
    assert (lens.cpu().numpy() <= 3).all()
