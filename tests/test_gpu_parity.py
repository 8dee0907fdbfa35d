"""GPU parity: the CUDA library against the CPU oracle, bit for bit, through the C-ABI binding."""
import numpy as np
import pytest

import oracle
import workloads
from helpers import OracleBatch, describe_diff

pytestmark = pytest.mark.gpu


def run_workload(w, check_steps, rows=None, cache=True, fused_every=0, check_prefix_mask=True, dfa=True, **state_kw):
    """Feed the workload through the library and the oracle; compare statuses every step and
    masks (all rows in `rows`) at the steps in `check_steps`.  Returns the library's stats."""
    import torch

    import paper_2506_01151_b200 as fmt

    dev = torch.device("cuda:0")
    g = fmt.Grammar(w.ebnf, w.start, w.vocab, w.eos, dfa=dfa)
    st = fmt.State(g, w.batch, cache=cache, **state_kw)
    ob = OracleBatch(w)
    rows = list(range(w.batch)) if rows is None else rows
    Wm = g.mask_words
    mask = torch.zeros((w.batch, Wm), dtype=torch.int32, device=dev)
    status = torch.zeros(w.batch, dtype=torch.int32, device=dev)

    def advance(tokens):
        tok = torch.from_numpy(np.ascontiguousarray(tokens, dtype=np.int32)).to(dev)
        st.advance(tok, status)
        got = status.cpu().numpy()
        for b in range(w.batch):
            want = ob.advance(b, int(tokens[b]))
            assert got[b] == want, ("status", b, int(tokens[b]), w.vocab[int(tokens[b])] if tokens[b] >= 0 else None, got[b], want)

    def compare(tag):
        st.fill_mask(mask)
        got = mask.cpu().numpy().view(np.uint32)
        for b in rows:
            want = ob.mask(b)
            assert np.array_equal(got[b], want), (tag, b, describe_diff(w, got[b], want))

    for p in range(w.prefix.shape[0]):
        advance(w.prefix[p])
    if check_prefix_mask:
        compare("after prefix")
    for i in range(w.steps):
        r = np.nonzero(w.reset_before[i])[0]
        if len(r):
            st.reset(torch.from_numpy(r.astype(np.int32)).to(dev))
            for b in r:
                ob.reset(int(b))
        advance(w.tokens[i])
        if i in check_steps:
            compare("step %d" % i)
            if fused_every and (i % fused_every == 0):
                logits = workloads.f32_to_bf16_bits(w.logits_f32(i))
                lt = torch.from_numpy(logits.view(np.int16)).to(dev)
                m2 = torch.zeros_like(mask)
                st.fill_and_apply(lt, fmt.BF16, mask_dev=m2)
                want_mask = np.stack([ob.mask(b) for b in range(w.batch)])
                assert np.array_equal(m2.cpu().numpy().view(np.uint32), want_mask)
                want = oracle.apply_mask(want_mask, logits, "bf16")
                assert np.array_equal(lt.cpu().numpy().view(np.uint16), want)
    q = st.query()
    for b in range(w.batch):
        assert bool(q["accepting"][b]) == ob.seqs[b].accepting, b
        assert bool(q["finished"][b] == 1) == ob.finished[b], b
    stats = st.stats()
    assert stats["capacity_errors"] == 0
    return stats, q


def test_config1_every_step():
    w = workloads.build(1)
    stats, _ = run_workload(w, check_steps=set(range(w.steps)), fused_every=4)
    assert stats["fills_computed"] > 0


def test_config1_without_cache():
    w = workloads.build(1)
    stats, q = run_workload(w, check_steps=set(range(w.steps)), cache=False)
    assert stats["fills_from_cache"] == 0 and (q["state_id"] == -1).all()


# Every reduced case runs both ways: each row swept from its own chart (the default), and with the
# cache of context-independent entries (Section 4.3) that lets rows share table look-ups.
BOTH_WAYS = pytest.mark.parametrize("roots", [False, True], ids=["from_chart", "ci_cache"])


@BOTH_WAYS
def test_config2_small_vocab_every_step(roots):
    w = workloads.build(2, V=4000, batch=4, steps=96)
    stats, _ = run_workload(w, check_steps=set(range(w.steps)), fused_every=16, roots=roots)
    assert (stats["roots"] > 0) == roots and (stats["rows_from_root"] + stats["rows_mask_only"] > 0) == roots


def test_config2_full():
    w = workloads.build(2)
    stats, _ = run_workload(w, check_steps=set(range(0, w.steps, 8)) | {w.steps - 1}, fused_every=64)
    assert stats["fills_from_cache"] + stats["fills_shared"] > 0  # pruned charts repeat (state cache)


@BOTH_WAYS
def test_config3_reduced(roots):
    w = workloads.build(3, V=20000, batch=8, steps=160)
    run_workload(w, check_steps=set(range(0, 160, 8)), fused_every=40, roots=roots)


@BOTH_WAYS
def test_config4_reduced(roots):
    w = workloads.build(4, V=20000, batch=8, steps=128)
    run_workload(w, check_steps=set(range(0, 128, 8)), fused_every=32, roots=roots)


@BOTH_WAYS
def test_config5_reduced(roots):
    w = workloads.build(5, V=20000, batch=8, steps=32, prefix_scale=0.25)
    run_workload(w, check_steps=set(range(0, 32, 4)), fused_every=16, roots=roots)


@pytest.mark.parametrize("config", [2, 3, 4, 5])
def test_reduced_configs_with_every_non_terminal_kept_as_rules(config):
    """By default regular non-terminals run as automata (Section 4.1); with that switched off the
    same masks must come out of rules alone."""
    kw = {2: dict(V=4000, batch=4, steps=64), 3: dict(V=20000, batch=8, steps=96), 4: dict(V=20000, batch=8, steps=64),
          5: dict(V=20000, batch=8, steps=24, prefix_scale=0.25)}[config]
    w = workloads.build(config, **kw)
    run_workload(w, check_steps=set(range(0, w.steps, 4)), fused_every=16, dfa=False)


# ---- full sizes, in the launch configuration the benchmark times; masks compared on sampled steps


def _sampled(steps, every):
    return set(range(0, steps, every)) | set(range(4)) | set(range(steps - 4, steps))


def test_config3_full_size_sampled_steps():
    w = workloads.build(3)
    stats, _ = run_workload(w, check_steps=_sampled(w.steps, 16), fused_every=128, check_prefix_mask=False)
    assert stats["fills_from_cache"] > stats["fills_computed"]  # the state cache carries most fills


def test_config4_full_size_sampled_steps():
    w = workloads.build(4)
    run_workload(w, check_steps=_sampled(w.steps, 16), fused_every=128, check_prefix_mask=False)


def test_config3_full_size_with_the_context_independent_cache():
    w = workloads.build(3, steps=192)
    stats, _ = run_workload(w, check_steps=_sampled(w.steps, 24), check_prefix_mask=False, roots=True)
    assert stats["rows_from_root"] + stats["rows_mask_only"] > 0.8 * stats["fills_computed"] and stats["root_sweeps"] > 0
    assert stats["fills_aborted"] == 0


def test_config5_full_size_sampled_rows_and_steps():
    w = workloads.build(5)
    rows = list(range(0, w.batch, 16))
    stats, q = run_workload(w, check_steps=set(range(0, w.steps, 4)), rows=rows, check_prefix_mask=False)
    assert q["n_sets"].max() > 20  # deep nesting / ambiguous segments keep many sets alive
