"""Pins for the oracle's suffix-trie store (Section 3, "Suffix Tree
Construction"; COUNT as defined below Eq. 2)."""
import numpy as np
import pytest

from bruteforce import distinct_substrings, occurrences


def _random_seqs(rng, n_seqs, lo, hi, vocab):
    return [rng.integers(0, vocab, size=int(rng.integers(lo, hi + 1))).tolist() for _ in range(n_seqs)]


@pytest.mark.parametrize("D", [1, 3, 5, 32])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_counts_equal_bruteforce_occurrences(oracle_mod, D, seed):
    rng = np.random.default_rng(seed)
    seqs = _random_seqs(rng, 4, 1, 14, 3)
    o = oracle_mod.SuffixOracle(D, 1)
    for s in seqs:
        o.global_insert(s)
    subs = distinct_substrings(seqs, D)
    # the trie holds exactly the distinct substrings of length <= D ...
    assert o.node_count(-1) == len(subs)
    # ... and each node's COUNT is its number of occurrences
    for path in subs:
        assert o.count(-1, path) == occurrences(seqs, path)
    # a string that does not occur has no node
    assert o.count(-1, [7]) == 0
    depth, parent, tok, cnt = o.dump(-1)
    paths = {}
    for i in range(len(tok)):
        paths[i] = (paths[parent[i]] if parent[i] >= 0 else ()) + (int(tok[i]),)
        assert depth[i] == len(paths[i])
        assert cnt[i] == occurrences(seqs, paths[i])
    assert set(paths.values()) == subs


def test_closed_form_single_repeated_token(oracle_mod):
    # corpus a^L: one chain, COUNT at depth d is L - d + 1
    L, D = 20, 8
    o = oracle_mod.SuffixOracle(D, 1)
    o.global_insert([4] * L)
    assert o.node_count(-1) == D
    for d in range(1, D + 1):
        assert o.count(-1, [4] * d) == L - d + 1
    assert o.count(-1, [4] * (D + 1)) == 0


def test_closed_form_all_distinct_and_k_copies(oracle_mod):
    L, D, k = 12, 5, 3
    seq = list(range(100, 100 + L))
    o = oracle_mod.SuffixOracle(D, 1)
    o.global_insert(seq)
    assert o.node_count(-1) == sum(L - d + 1 for d in range(1, D + 1))
    _, _, _, cnt = o.dump(-1)
    assert (cnt == 1).all()
    for _ in range(k - 1):
        o.global_insert(seq)
    _, _, _, cnt = o.dump(-1)
    assert (cnt == k).all()


def test_sequences_do_not_join(oracle_mod):
    o = oracle_mod.SuffixOracle(4, 1)
    o.global_insert([1, 2])
    o.global_insert([3, 4])
    assert o.count(-1, [2, 3]) == 0
    assert o.count(-1, [1, 2]) == 1


@pytest.mark.parametrize("seed", [3, 4])
def test_count_invariants(oracle_mod, seed):
    rng = np.random.default_rng(seed)
    D = 4
    seqs = _random_seqs(rng, 5, 2, 12, 3)
    o = oracle_mod.SuffixOracle(D, 1)
    for s in seqs:
        o.global_insert(s)
    depth, parent, tok, cnt = o.dump(-1)
    n_tokens = sum(len(s) for s in seqs)
    assert cnt[parent == -1].sum() == n_tokens
    paths = {}
    child_sum = np.zeros(len(tok), dtype=np.int64)
    for i in range(len(tok)):
        paths[i] = (paths[parent[i]] if parent[i] >= 0 else ()) + (int(tok[i]),)
        if parent[i] >= 0:
            child_sum[parent[i]] += cnt[i]
    for i in range(len(tok)):
        p = list(paths[i])
        if depth[i] == D:
            assert child_sum[i] == 0
        else:
            ends = sum(1 for s in seqs if len(s) >= len(p) and s[len(s) - len(p):] == p)
            assert cnt[i] - child_sum[i] == ends


@pytest.mark.parametrize("D", [2, 4, 32])
def test_incremental_equals_from_scratch(oracle_mod, D):
    rng = np.random.default_rng(11)
    text = rng.integers(0, 3, size=40).tolist()
    inc = oracle_mod.SuffixOracle(D, 1)
    for t in range(1, len(text) + 1):
        inc.slot_append(0, [text[t - 1]])
        if t in (1, 2, 5, 17, 40):
            ref = oracle_mod.SuffixOracle(D, 1)
            ref.global_insert(text[:t])
            a, b = inc.dump(0), ref.dump(-1)
            for x, y in zip(a, b):
                assert np.array_equal(x, y)
            for path in distinct_substrings([text[:t]], D):
                assert inc.count(0, path) == occurrences([text[:t]], path)
    assert np.array_equal(inc.slot_text(0), np.asarray(text, dtype=np.int32))
    inc.slot_reset(0)
    assert inc.node_count(0) == 0 and inc.slot_len(0) == 0


def test_append_in_chunks_equals_token_by_token(oracle_mod):
    rng = np.random.default_rng(5)
    text = rng.integers(0, 4, size=60).tolist()
    a = oracle_mod.SuffixOracle(6, 2)
    a.slot_append(0, text)
    a.slot_append_batch([1], [text[:25]], n_threads=2)
    a.slot_append_batch([1], [text[25:]], n_threads=2)
    for x, y in zip(a.dump(0), a.dump(1)):
        assert np.array_equal(x, y)


def test_entropy_closed_forms_and_bruteforce(oracle_mod):
    """Appendix "Predicting SuffixDecoding Effectiveness": count-weighted mean of the entropy of
    every node's children distribution (bits)."""
    import math
    from bruteforce import children
    # sequences [a,b], [a,c]: root {a:2, b:1, c:1} -> 1.5 bits, weight 4; node a {b:1, c:1} -> 1 bit, weight 2
    o = oracle_mod.SuffixOracle(4, 1)
    o.global_insert([1, 2]); o.global_insert([1, 3])
    assert abs(o.entropy(-1) - (4 * 1.5 + 2 * 1.0) / 6) < 1e-12
    # one repeated token: every node has a single child -> 0
    o = oracle_mod.SuffixOracle(6, 1)
    o.global_insert([7] * 15)
    assert o.entropy(-1) == 0.0
    assert oracle_mod.SuffixOracle(6, 1).entropy(-1) == 0.0      # empty tree
    # k equally likely tokens, depth cap 1: log2 k
    o = oracle_mod.SuffixOracle(1, 1)
    o.global_insert(list(range(8)) * 3)
    assert abs(o.entropy(-1) - 3.0) < 1e-12
    # brute force from substring scans on a random corpus
    rng = np.random.default_rng(17)
    D = 4
    seqs = [rng.integers(0, 3, size=int(rng.integers(3, 14))).tolist() for _ in range(4)]
    o = oracle_mod.SuffixOracle(D, 1)
    for s in seqs:
        o.global_insert(s)
    acc = weight = 0.0
    stack = [[]]
    while stack:
        path = stack.pop()
        ch = children(seqs, path, D)
        tot = sum(ch.values())
        if tot:
            acc += tot * -sum(c / tot * math.log2(c / tot) for c in ch.values())
            weight += tot
            stack.extend(path + [t] for t in ch)
    assert abs(o.entropy(-1) - acc / weight) < 1e-12
