"""GPU edge cases through the C-ABI binding: statuses, EOS, odd vocabularies, logits layouts,
cache limits, the large-scratch paths and capacity errors.  Expected values come from the CPU
oracle or from the definition of the operation."""
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


def test_statuses_eos_and_odd_vocabulary():
    import paper_2506_01151_b200 as fmt

    # duplicates, an empty non-EOS token, a token no sentence contains, EOS in the middle of the ids
    vocab = [b"a", b"b", b"", b"ab", b"a", b"", b"zz", b"ba"]
    eos = 5
    text = 's ::= "a" s "b" | "ab"'
    g = fmt.Grammar(text, "s", vocab, eos)
    og, ov = oracle.Grammar(text, "s"), oracle.Vocab(vocab, eos)
    st = fmt.State(g, 4)
    seqs = [oracle.Sequence_(og) for _ in range(4)]

    def check():
        got = _mask_of(st, g, 4)
        for b in range(4):
            assert np.array_equal(got[b], seqs[b].mask(ov)), b

    check()
    # row 0: "a" ok; row 1: "b" rejected; row 2: empty token rejected; row 3: skipped
    assert _advance(st, [0, 1, 2, -1]) == [fmt.FMT_OK, fmt.ERR_TOKEN_REJECTED, fmt.ERR_TOKEN_REJECTED, fmt.FMT_OK]
    seqs[0].advance(b"a")
    check()
    # out-of-range ids; EOS while not accepting; duplicate id 4 == "a"
    assert _advance(st, [99, -5, eos, 4]) == [fmt.ERR_INVALID_ARG, fmt.ERR_INVALID_ARG, fmt.ERR_TOKEN_REJECTED, fmt.FMT_OK]
    seqs[3].advance(b"a")
    check()
    # finish rows 0 and 3 ("aabb" / "ab"), then EOS
    assert _advance(st, [3, -1, -1, 1]) == [0, 0, 0, 0]
    seqs[0].advance(b"ab")
    seqs[3].advance(b"b")
    check()
    assert _advance(st, [1, -1, -1, eos]) == [0, 0, 0, 0]
    seqs[0].advance(b"b")
    got = _mask_of(st, g, 4)
    assert np.array_equal(got[0], seqs[0].mask(ov)) and got[0][0] == 1 << eos  # only EOS may follow "aabb"
    assert got[3][0] == 1 << eos  # finished: the EOS bit alone
    assert _advance(st, [eos, -1, -1, 0]) == [0, 0, 0, fmt.ERR_FINISHED]
    q = st.query()
    assert q["finished"].tolist() == [1, 0, 0, 1] and q["accepting"].tolist()[0] == 1
    # reset brings a finished row back
    torch, dev = _torch()
    st.reset(torch.tensor([3], dtype=torch.int32, device=dev))
    seqs[3] = oracle.Sequence_(og)
    got = _mask_of(st, g, 4)
    assert np.array_equal(got[3], seqs[3].mask(ov))


def test_nullable_start_and_empty_sentence():
    import paper_2506_01151_b200 as fmt

    text = 's ::= item*\nitem ::= "x" | "(" s ")"'
    vocab = [b"x", b"(", b")", b"()", b"(x", b"))", b""]
    g = fmt.Grammar(text, "s", vocab, 6)
    assert g.info().start_nullable == 1
    og, ov = oracle.Grammar(text, "s"), oracle.Vocab(vocab, 6)
    st = fmt.State(g, 1)
    seq = oracle.Sequence_(og)
    rng = np.random.default_rng(3)
    for step in range(60):
        got = _mask_of(st, g, 1)[0]
        want = seq.mask(ov)
        assert np.array_equal(got, want), step
        choices = [t for t in range(6) if (want[0] >> t) & 1]
        t = int(rng.choice(choices))
        assert _advance(st, [t]) == [0]
        assert seq.advance(vocab[t])


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_apply_mask_layouts_and_special_values(dtype):
    import paper_2506_01151_b200 as fmt

    torch, dev = _torch()
    rng = np.random.default_rng(11)
    B, V = 5, 1003  # V not a multiple of 8 or 32
    words, stride_words, row_stride = (V + 31) // 32, (V + 31) // 32 + 3, V + 5  # odd row stride: unaligned rows
    mask = rng.integers(0, 2**32, size=(B, stride_words), dtype=np.uint64).astype(np.uint32)
    mask[1, :] = 0
    mask[2, :] = 0xFFFFFFFF
    f = rng.standard_normal((B, row_stride)).astype(np.float32)
    f[0, 3], f[1, 5], f[2, 7], f[3, 9], f[4, 11] = np.nan, np.inf, -np.inf, -0.0, np.nan
    if dtype == "bf16":
        host = workloads.f32_to_bf16_bits(f)
        host[0, 13] = 0x7FC1  # NaN with a payload
        dev_t = torch.from_numpy(host.view(np.int16)).to(dev)
        code = fmt.BF16
    else:
        host = f.copy()
        dev_t = torch.from_numpy(host).to(dev)
        code = fmt.FP32
    m_t = torch.from_numpy(mask.view(np.int32)).to(dev)
    fmt.apply_mask(m_t, dev_t, code, B, V, stride_words=stride_words, row_stride=row_stride)
    got = dev_t.cpu().numpy()
    got = got.view(np.uint16) if dtype == "bf16" else got
    want = host.copy()
    want[:, :V] = oracle.apply_mask(np.ascontiguousarray(mask[:, :words]), np.ascontiguousarray(host[:, :V]), dtype)
    if dtype == "bf16":
        assert np.array_equal(got, want)
    else:
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))  # padding beyond V untouched as well


def test_fused_apply_fp32_and_wide_mask_stride():
    import paper_2506_01151_b200 as fmt

    torch, dev = _torch()
    w = workloads.build(1)
    g = fmt.Grammar(w.ebnf, w.start, w.vocab, w.eos)
    st = fmt.State(g, 1)
    og, ov = oracle.Grammar(w.ebnf, w.start), oracle.Vocab(w.vocab, w.eos)
    seq = oracle.Sequence_(og)
    for p in range(w.prefix.shape[0]):
        assert _advance(st, [int(w.prefix[p, 0])]) == [0]
    seq.advance(w.prefix_bytes[0])
    logits = w.logits_f32(0)
    lt = torch.from_numpy(logits.copy()).to(dev)
    stride = g.mask_words + 4
    m = torch.full((1, stride), -1, dtype=torch.int32, device=dev)
    st.fill_and_apply(lt, fmt.FP32, mask_dev=m, stride_words=stride)
    want_mask = seq.mask(ov)[None, :]
    got_mask = m.cpu().numpy().view(np.uint32)
    assert np.array_equal(got_mask[:, : g.mask_words], want_mask) and not got_mask[:, g.mask_words:].any()
    want = oracle.apply_mask(want_mask, logits, "fp32")
    assert np.array_equal(lt.cpu().numpy().view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("keep", [True, False], ids=["keep_when_full", "empty_when_full"])
def test_tiny_cache_still_gives_right_masks(keep):
    """A state cache far too small for the workload: either it keeps its first entries and takes no
    more (rows that found no room carry their charts themselves), or - the default - it is emptied
    whenever it has no room left and goes on caching.  The masks are the oracle's either way."""
    import paper_2506_01151_b200 as fmt

    torch, dev = _torch()
    w = workloads.build(2, V=3000, batch=4, steps=60)
    g = fmt.Grammar(w.ebnf, w.start, w.vocab, w.eos)
    st = fmt.State(g, w.batch, max_states=8, max_mask_rows=2, pool_words=4096, keep_when_full=keep)  # fills up at once
    og, ov = oracle.Grammar(w.ebnf, w.start), oracle.Vocab(w.vocab, w.eos)
    seqs = [oracle.Sequence_(og) for _ in range(w.batch)]
    for p in range(w.prefix.shape[0]):
        _advance(st, [int(x) for x in w.prefix[p]])
    for b in range(w.batch):
        seqs[b].advance(w.prefix_bytes[b])
    for i in range(w.steps):
        r = np.nonzero(w.reset_before[i])[0]
        if len(r):
            st.reset(torch.from_numpy(r.astype(np.int32)).to(dev))
        assert _advance(st, [int(x) for x in w.tokens[i]]) == [0] * w.batch
        fin = [False] * w.batch
        for b in range(w.batch):
            if w.reset_before[i, b]:
                seqs[b] = oracle.Sequence_(og)
            t = int(w.tokens[i, b])
            if t == w.eos:
                fin[b] = True
            else:
                seqs[b].advance(w.vocab[t])
        if i % 6 == 0:
            got = _mask_of(st, g, w.batch)
            for b in range(w.batch):
                if not fin[b]:
                    assert np.array_equal(got[b], seqs[b].mask(ov)), (i, b)
    s = st.stats()
    assert s["states_cached"] <= 8 and s["mask_rows_cached"] <= 2 and s["capacity_errors"] == 0
    if keep:
        assert s["cache_flushes"] == 0
        assert (st.query()["state_id"] == -1).any()  # some rows could not be cached and carry their chart themselves
    else:
        assert s["cache_flushes"] >= 3  # emptied again and again, and entries taken again after each time
        assert s["fills_from_cache"] + s["advances_cached"] >= 0


def _wide_grammar(n):
    # one alternation of n literals with a shared first byte: Earley sets of several thousand items
    rng = np.random.default_rng(5)
    names = set()
    while len(names) < n:
        names.add("k" + "".join(rng.choice(list("abcdefgh"), size=6)))
    names = sorted(names)
    text = 's ::= "[" name ( "," name )* "]"\nname ::= ' + " | ".join('"%s"' % x for x in names)
    return text, names


def test_sets_larger_than_shared_memory_use_the_large_scratch():
    import paper_2506_01151_b200 as fmt

    text, names = _wide_grammar(1500)
    vocab = [bytes([b]) for b in range(256)] + [b"[k", b"ka", b"kb", b",k", names[0].encode(), names[7][:4].encode(),
                                                 (names[3] + ",").encode(), b"]", b"kab", b""]
    eos = len(vocab) - 1
    g = fmt.Grammar(text, "s", vocab, eos)
    og, ov = oracle.Grammar(text, "s"), oracle.Vocab(vocab, eos)
    st = fmt.State(g, 2)
    seqs = [oracle.Sequence_(og) for _ in range(2)]
    feeds = [[b"[k", names[5][1:].encode(), b","], [b"[", b"k", names[9][1:3].encode()]]
    index = {t: i for i, t in enumerate(vocab)}
    for step in range(3):
        toks = []
        for b in range(2):
            data = feeds[b][step]
            if data in index:
                toks.append([index[data]])
            else:
                toks.append([index[bytes([c])] for c in data])
        for k in range(max(len(t) for t in toks)):
            ids = [t[k] if k < len(t) else -1 for t in toks]
            assert _advance(st, ids) == [0, 0]
        for b in range(2):
            assert seqs[b].advance(feeds[b][step])
        got = _mask_of(st, g, 2)
        for b in range(2):
            assert np.array_equal(got[b], seqs[b].mask(ov)), (step, b)
    s = st.stats()
    assert s["capacity_errors"] == 0
    assert s["big_mode_units"] > 0  # the sweep met sets beyond its shared-memory scratch
    assert s["chart_items_max"] > 1000


def test_capacity_overflow_is_reported_not_guessed():
    import paper_2506_01151_b200 as fmt

    text, names = _wide_grammar(1500)
    vocab = [bytes([b]) for b in range(256)] + [b""]
    g = fmt.Grammar(text, "s", vocab, 256)
    st = fmt.State(g, 2, chart_words=1024)  # far too small for a chart with 1500 predicted items
    assert _advance(st, [ord("["), -1]) == [fmt.ERR_CAPACITY, fmt.FMT_OK]
    got = _mask_of(st, g, 2)
    assert not got[0].any()  # the broken row's mask is all-zero
    og, ov = oracle.Grammar(text, "s"), oracle.Vocab(vocab, 256)
    assert np.array_equal(got[1], oracle.Sequence_(og).mask(ov))  # the other row is unaffected
    assert _advance(st, [ord("k"), ord("[")]) == [fmt.ERR_CAPACITY, fmt.ERR_CAPACITY]
    assert st.query()["finished"].tolist() == [2, 2]
    assert st.stats()["capacity_errors"] >= 2
    # a state with too few walk states reports the capacity problem through the mask (all-zero) as well
    st2 = fmt.State(g, 1, sweep_states=16)
    assert _advance(st2, [ord("[")]) == [0]
    for c in names[0].encode():
        assert _advance(st2, [c]) == [0]
    seq = oracle.Sequence_(og)
    assert seq.advance(b"[" + names[0].encode())
    got2 = _mask_of(st2, g, 1)[0]
    if st2.stats()["capacity_errors"]:
        assert not got2.any()  # reported: the mask is all-zero, never a partial one
    else:
        assert np.array_equal(got2, seq.mask(ov))


def test_sweep_hash_generations_start_over():
    """The sweep's per-job hashes of Earley sets are never cleared between fills: every fill has a
    16-bit generation (two per fill: one for the sweep of new roots, one for the rows' own walks) and
    takes slots of other generations for empty.  When the numbers start over (every 32767 fills) the
    tables are cleared first, or a fill would meet its own old entries.  Two rows with the state cache
    off (every fill computes them) go through more than 65535 fills; the masks before, at and after
    every turn must equal the oracle's."""
    import paper_2506_01151_b200 as fmt

    torch, dev = _torch()
    w = workloads.build(1, steps=4)
    g = fmt.Grammar(w.ebnf, w.start, w.vocab, w.eos)
    og, ov = oracle.Grammar(w.ebnf, w.start), oracle.Vocab(w.vocab, w.eos)
    st = fmt.State(g, 2, cache=False)
    seqs = [oracle.Sequence_(og) for _ in range(2)]
    for b, text in enumerate([b"(1+", b"12*(3"]):
        toks = [w.vocab.index(bytes([c])) for c in text]  # the single bytes are tokens 0..255
        for t in toks:
            ids = [-1, -1]
            ids[b] = t
            assert _advance(st, ids)[b] == fmt.FMT_OK
        assert seqs[b].advance(text)
    want = np.stack([s.mask(ov) for s in seqs])
    m = torch.zeros((2, g.mask_words), dtype=torch.int32, device=dev)
    total = 65535 + 40
    for i in range(total):
        st.fill_mask(m)
        if i in (0, 32765, 32766, 32767, 32768, 32769, 65532, 65533, 65534, 65535, 65536, total - 1):
            assert np.array_equal(m.cpu().numpy().view(np.uint32), want), i
    assert st.stats()["capacity_errors"] == 0


def test_advance_transition_cache_replays_exactly():
    """Advancing a cached chart by a token it has been advanced by before is answered from the
    transition cache.  The same token streams are fed twice (rows reset in between) with a
    rejected token slipped in: statuses, masks, charts and cache ids of the second pass, which
    runs no Earley step, must equal those of the first, and the masks the oracle's."""
    import paper_2506_01151_b200 as fmt
    from helpers import OracleBatch

    torch, dev = _torch()
    w = workloads.build(2, V=6000, batch=4, steps=20)
    g = fmt.Grammar(w.ebnf, w.start, w.vocab, w.eos)
    st = fmt.State(g, w.batch)
    bad = ord("}")  # ids 0..255 are the single bytes; "}" cannot open a JSON document

    def run():
        ob = OracleBatch(w)
        st.reset()
        seen = []
        assert _advance(st, [bad] * w.batch) == [fmt.ERR_TOKEN_REJECTED] * w.batch
        for p in range(w.prefix.shape[0]):
            toks = w.prefix[p].tolist()
            want = [ob.advance(b, t) for b, t in enumerate(toks)]
            assert _advance(st, toks) == want
        for i in range(w.steps):
            if w.reset_before[i].any():
                break
            toks = w.tokens[i].tolist()
            want = [ob.advance(b, t) for b, t in enumerate(toks)]
            assert _advance(st, toks) == want, i
            got = _mask_of(st, g, w.batch)
            for b in range(w.batch):
                assert np.array_equal(got[b], ob.mask(b)), (i, b)
            q = st.query()
            seen.append((got.copy(), [st.chart_words(b).tolist() for b in range(w.batch)], list(q["state_id"])))
        return seen

    first = run()
    s0 = st.stats()
    second = run()
    s1 = st.stats()
    assert len(first) == len(second) and len(first) > 4
    for a, b in zip(first, second):
        assert np.array_equal(a[0], b[0]) and a[1] == b[1] and a[2] == b[2]
    replayed = s1["steps_advanced"] - s0["steps_advanced"]
    assert replayed > 0 and s1["advances_cached"] - s0["advances_cached"] == replayed
    assert s1["states_cached"] == s0["states_cached"]


def test_entries_in_use_survive_when_the_cache_turns_over():
    """A cache of 8 entries; row 1 meets a new chart at every step (right recursion keeps its history), row 0
    is sent back to the start at every step.  The cache fills up and is turned over again and again; the start
    state, found again every time, must keep its mask through every turn-over: it is computed exactly once."""
    import paper_2506_01151_b200 as fmt

    torch, dev = _torch()
    text = 's ::= "a" s | "b"'
    vocab = [b"a", b"b", b"ab", b"aab", b""]
    g = fmt.Grammar(text, "s", vocab, 4, dfa=False)
    og, ov = oracle.Grammar(text, "s"), oracle.Vocab(vocab, 4)
    st = fmt.State(g, 2, max_states=8, max_mask_rows=8, pool_words=1 << 16)
    seq1 = oracle.Sequence_(og)
    start_mask = oracle.Sequence_(og).mask(ov)
    row0 = torch.tensor([0], dtype=torch.int32, device=dev)
    for i in range(40):
        assert _advance(st, [0, 0]) == [0, 0]  # both rows take "a"
        assert seq1.advance(b"a")
        st.reset(row0)
        got = _mask_of(st, g, 2)
        assert np.array_equal(got[0], start_mask) and np.array_equal(got[1], seq1.mask(ov)), i
    s = st.stats()
    assert s["cache_flushes"] >= 3 and s["capacity_errors"] == 0
    # 40 new charts for row 1, and the start state once (its first fill): every other fill of row 0 was a hit
    assert s["fills_computed"] == 41, s["fills_computed"]
    assert s["fills_from_cache"] == 39
