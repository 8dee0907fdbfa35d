"""The allocation-free entry point, fmt_fill_mask_noalloc, against the CPU oracle and fmt_fill_mask.

Some callers may not allocate device memory while they run (all memory handed out up front, an
allocation could synchronize the device or fail under pressure), so they cannot create an
fmt_state.  For them the library computes masks for charts they already hold, using a scratch
array built into the library image.  Here the charts come from an ordinary fmt_state; the two
entry points must agree with the oracle's masks bit for bit, on two calls in a row (the second call meets the scratch
array as the first one left it).  This file is collected last on purpose.
"""
import numpy as np
import pytest

import workloads
from helpers import OracleBatch

pytestmark = pytest.mark.gpu


def test_noalloc_matches_fill_mask_on_two_calls_in_a_row():
    import torch

    import paper_2506_01151_b200 as fmt

    dev = torch.device("cuda:0")
    w = workloads.build(2, V=6000, batch=6, steps=40)
    g = fmt.Grammar(w.ebnf, w.start, w.vocab, w.eos)
    st = fmt.State(g, w.batch)
    ob = OracleBatch(w)
    status = torch.zeros(w.batch, dtype=torch.int32, device=dev)
    for p in range(w.prefix.shape[0]):
        st.advance(torch.from_numpy(w.prefix[p].copy()).to(dev), status)
        for b in range(w.batch):
            ob.advance(b, int(w.prefix[p][b]))
    Wm = g.mask_words
    want = torch.zeros((w.batch, Wm), dtype=torch.int32, device=dev)
    calls = 0
    for i in range(w.steps):
        r = np.nonzero(w.reset_before[i])[0]
        if len(r):
            st.reset(torch.from_numpy(r.astype(np.int32)).to(dev))
            for b in r:
                ob.reset(int(b))
        st.advance(torch.from_numpy(w.tokens[i].copy()).to(dev), status)
        for b in range(w.batch):
            ob.advance(b, int(w.tokens[i][b]))
        if i not in (7, 8, 30):  # two calls in a row, then one more later
            continue
        st.fill_mask(want)
        q = st.query()
        rows = [b for b in range(w.batch) if q["finished"][b] == 0]  # finished rows have no chart semantics
        charts = [st.chart_words(b) for b in rows]
        offs = np.zeros(len(rows) + 1, dtype=np.uint64)
        offs[1:] = np.cumsum([len(c) + 5 for c in charts])  # a little slack after each chart
        blob = np.zeros(int(offs[-1]), dtype=np.uint32)
        for c, o in zip(charts, offs[:-1]):
            blob[int(o):int(o) + len(c)] = c
        charts_dev = torch.from_numpy(blob.view(np.int32)).to(dev)
        got = torch.full((len(rows), Wm), -1, dtype=torch.int32, device=dev)  # must be overwritten entirely
        st2 = torch.full((len(rows),), -1, dtype=torch.int32, device=dev)
        fmt.fill_mask_noalloc(g, charts_dev, offs, got, st2)
        torch.cuda.synchronize()
        assert (st2.cpu().numpy() == 0).all()
        oracle_masks = np.stack([ob.mask(b) for b in rows])
        assert np.array_equal(got.cpu().numpy().view(np.uint32), oracle_masks), "call %d differs from the oracle" % calls
        assert np.array_equal(got.cpu().numpy(), want.cpu().numpy()[rows]), "call %d differs" % calls
        assert got.cpu().numpy().any()
        calls += 1
    assert calls == 3


def test_noalloc_rejects_what_does_not_fit():
    import torch

    import paper_2506_01151_b200 as fmt

    dev = torch.device("cuda:0")
    g = fmt.Grammar('s ::= "a" s | "b"', "s", [b"a", b"b", b"ab", b""], 3)
    st = fmt.State(g, 1)
    chart = st.chart_words(0)
    charts_dev = torch.from_numpy(chart.view(np.int32)).to(dev)
    mask = torch.zeros((65, g.mask_words), dtype=torch.int32, device=dev)
    with pytest.raises(fmt.FmtError) as e:  # more charts than the fixed scratch is laid out for
        fmt.fill_mask_noalloc(g, charts_dev, [0] * 66, mask)
    assert e.value.code == fmt.ERR_CAPACITY and "64" in str(e.value)
    # a slot smaller than the chart's header claims: reported per chart, mask left all-zero
    status = torch.full((2,), -1, dtype=torch.int32, device=dev)
    fmt.fill_mask_noalloc(g, charts_dev, [0, len(chart) - 1, len(chart) - 1], mask, status)
    torch.cuda.synchronize()
    assert status.cpu().numpy().tolist() == [fmt.ERR_INVALID_ARG, fmt.ERR_INVALID_ARG]
    assert not mask.cpu().numpy()[:2].any()
    # and the intact chart still works afterwards: a, b, ab valid at the start, EOS not
    fmt.fill_mask_noalloc(g, charts_dev, [0, len(chart)], mask, status)
    torch.cuda.synchronize()
    assert status.cpu().numpy()[0] == 0 and mask.cpu().numpy()[0, 0] == 0b0111


def test_noalloc_checks_every_word_of_a_chart():
    """A chart whose header is fine but whose contents are not (offsets that decrease, an item that
    names a dotted rule or an origin set that does not exist) is reported and not swept; the intact
    chart beside it gets its mask."""
    import torch

    import paper_2506_01151_b200 as fmt

    dev = torch.device("cuda:0")
    g = fmt.Grammar('s ::= "a" s | "b"', "s", [b"a", b"b", b"ab", b""], 3)
    st = fmt.State(g, 1)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    st.advance(torch.tensor([0], dtype=torch.int32, device=dev), status)  # "a": a chart with more than one set
    good = st.chart_words(0).copy()
    hdr, m, items = 8, int(good[0]), int(good[1])  # header words; sets; items (the layout fmt_state_copy_chart documents)
    assert m >= 2 and len(good) == hdr + m + 1 + items
    first_item = hdr + m + 1
    n_dotted = g.info().n_dotted
    bad_rule = good.copy()
    bad_rule[first_item] = (int(bad_rule[first_item]) & 0xFFFF0000) | (n_dotted + 3)
    bad_origin = good.copy()
    bad_origin[first_item] = (m << 16) | (int(bad_origin[first_item]) & 0xFFFF)
    bad_offsets = good.copy()
    bad_offsets[hdr + 1] = items + 1  # set 0 would end beyond the last item, and after set 1 does
    blobs = [bad_rule, good, bad_origin, bad_offsets]
    offs = np.zeros(len(blobs) + 1, dtype=np.uint64)
    offs[1:] = np.cumsum([len(b) for b in blobs])
    charts_dev = torch.from_numpy(np.concatenate(blobs).view(np.int32)).to(dev)
    mask = torch.full((4, g.mask_words), -1, dtype=torch.int32, device=dev)
    status = torch.full((4,), -1, dtype=torch.int32, device=dev)
    fmt.fill_mask_noalloc(g, charts_dev, offs, mask, status)
    torch.cuda.synchronize()
    assert status.cpu().numpy().tolist() == [fmt.ERR_INVALID_ARG, 0, fmt.ERR_INVALID_ARG, fmt.ERR_INVALID_ARG]
    got = mask.cpu().numpy().view(np.uint32)
    assert not got[0].any() and not got[2].any() and not got[3].any()
    assert got[1, 0] == 0b0111  # after "a": a, b, ab
