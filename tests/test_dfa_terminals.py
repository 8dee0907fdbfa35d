"""Regular non-terminals compiled into automata (Section 4.1: terminals as regular languages run as
finite-state machines), checked on the host against the CPU oracle: the automaton of a non-terminal
must accept exactly the strings the oracle's Earley recognizer accepts with that non-terminal as the
start symbol.  Strings come from random walks through the automaton (accepted ones and ones cut
short), from single-byte corruptions of them, and from the workload's vocabulary."""
import numpy as np
import pytest

import oracle
import workloads
import paper_2506_01151_b200 as fmt


def _distance_to_accept(trans, accept, n_eq):
    """Per state, the fewest bytes to an accepting state."""
    S = len(accept)
    none = trans.reshape(S, n_eq) == 0xFFFF
    tgt = np.where(none, 0, trans.reshape(S, n_eq).astype(np.int64) & 0x3FFF)
    dist = np.where(np.asarray(accept) != 0, 0, 1 << 30).astype(np.int64)
    for _ in range(S + 1):
        via = np.where(none, 1 << 30, dist[tgt] + 1).min(axis=1)
        new = np.minimum(dist, via)
        if (new == dist).all():
            break
        dist = new
    return dist


def _walks(trans, accept, dist, start, n_eq, byte_of_class, rng, count, wander):
    """Walks from `start`: up to `wander` random steps, then the shortest way to an accepting state.
    Every string returned is accepted by the automaton."""
    out = []
    for _ in range(count):
        q, s = int(start), bytearray()
        steps = int(rng.integers(0, wander + 1))
        while True:
            row = trans[q * n_eq:(q + 1) * n_eq]
            live = np.nonzero(row != 0xFFFF)[0]
            if len(s) >= steps or len(live) == 0:
                if accept[q]:
                    break
                closer = [e for e in live if dist[int(row[e]) & 0x3FFF] < dist[q]]
                e = int(rng.choice(closer))
            else:
                e = int(rng.choice(live))
            s.append(int(rng.choice(byte_of_class[e])))
            q = int(row[e]) & 0x3FFF
        out.append(bytes(s))
    return out


def _oracle_accepts(og, data: bytes) -> bool:
    s = oracle.Sequence_(og)
    return s.advance(data) and s.accepting if data else s.accepting


@pytest.mark.parametrize("config", [1, 2, 3, 4, 5])
def test_each_automaton_accepts_what_the_oracle_accepts_for_its_nonterminal(config):
    w = workloads.build(config, V=2000, batch=1, steps=2, prefix_scale=0.05)
    g = fmt.Grammar(w.ebnf, w.start, w.vocab, w.eos, host_only=True)
    info = g.info()
    assert info.n_automata >= 1
    trans, accept, starts, cls = g.table(11), g.table(12), g.table(13), g.table(10)
    n_eq = info.n_byte_classes
    assert len(trans) == info.n_automaton_states * n_eq and len(accept) == info.n_automaton_states
    byte_of_class = [np.nonzero(cls == e)[0] for e in range(n_eq)]
    rng = np.random.default_rng(1151 + config)
    dist = _distance_to_accept(trans, accept, n_eq)
    assert (dist < (1 << 30)).all()  # every state can still reach an accepting one: nothing dead is kept
    checked = positives = 0
    for k in range(info.n_automata):
        name = g.automaton_name(k)
        if "~" in name:
            continue  # a helper made by the desugaring: the oracle's grammar has no non-terminal of that name
        og = oracle.Grammar(w.ebnf, name)
        cands = _walks(trans, accept, dist, starts[k], n_eq, byte_of_class, rng, 40, 30)
        for s in list(cands[:25]):  # single-byte corruptions and truncations
            if s:
                i = int(rng.integers(0, len(s)))
                cands.append(s[:i] + bytes([int(rng.integers(0, 256))]) + s[i + 1:])
                cands.append(s[:i])
        cands += [w.vocab[int(t)] for t in rng.integers(0, len(w.vocab) - 1, size=40)]
        cands.append(b"")
        for s in cands:
            want = _oracle_accepts(og, s)
            assert g.automaton_accepts(k, s) == want, (name, s)
            checked += 1
            positives += want
    assert checked >= 100 and positives >= 10, (checked, positives)


def test_what_is_not_regular_stays_rules():
    """Nested brackets are not a regular language; a list of digits is.  And the language as a whole
    is the same with and without the automata: compared on the oracle via the item tables' sizes and
    on enumerated strings via the automaton of the regular part."""
    text = 's ::= "(" s ")" | num\nnum ::= [0-9]+ ("." [0-9]+)?'
    vocab = [bytes([b]) for b in b"()0123456789."] + [b""]
    g = fmt.Grammar(text, "s", vocab, len(vocab) - 1, host_only=True)
    info = g.info()
    assert info.n_automata == 1 and g.automaton_name(0) == "num"
    assert g.automaton_accepts(0, b"12.5") and g.automaton_accepts(0, b"7")
    assert not g.automaton_accepts(0, b"12.") and not g.automaton_accepts(0, b".5") and not g.automaton_accepts(0, b"")
    g0 = fmt.Grammar(text, "s", vocab, len(vocab) - 1, host_only=True, dfa=False)
    assert g0.info().n_automata == 0 and g0.info().n_rules > info.n_rules
    # a grammar that is regular as a whole becomes one automaton
    g1 = fmt.Grammar('s ::= ("a" | "b" "c")* "d"', "s", [b"a", b""], 1, host_only=True)
    assert g1.info().n_automata == 1 and g1.info().n_rules == 1  # only $ -> s is left
    for s, ok in [(b"d", True), (b"abcd", True), (b"bcbcad", True), (b"abd", False), (b"", False), (b"dd", False)]:
        assert g1.automaton_accepts(0, s) == ok, s
