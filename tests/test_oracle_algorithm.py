"""Pins for the oracle's MatchPattern / ExpandSpeculationTree / SCORE /
GenerateCandidateTree (Algorithm 1, Eq. 1-4) and the hand-off arrays."""
import json
import os
from fractions import Fraction

import numpy as np
import pytest

from bruteforce import best_connected_score, greedy_tree, occurrences, subtree_nodes

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _mk(oracle_mod, D, seqs, n_slots=1):
    o = oracle_mod.SuffixOracle(D, n_slots)
    for s in seqs:
        o.global_insert(s)
    return o


def test_hand_worked_example(oracle_mod):
    g = json.load(open(os.path.join(GOLDEN, "hand_example.json")))
    o = _mk(oracle_mod, g["depth_cap"], g["global_sequences"])
    o.slot_append(0, g["context"])
    r = o.speculate([0], g["P"], g["alpha"], g["max_spec"])
    e = g["expected"]
    n = e["n_draft"]
    assert r["n_draft"][0] == n
    assert r["tokens"][0, :n].tolist() == e["tokens"]
    assert r["parents"][0, :n].tolist() == e["parents"]
    assert r["positions"][0, :n].tolist() == e["positions"]
    assert r["mask"][0, :n, 0].tolist() == e["mask_rows"]
    assert (r["tokens"][0, n:] == -1).all() and (r["mask"][0, n:] == 0).all()
    assert r["chosen_tree"][0] == e["chosen_tree"] and r["chosen_p"][0] == e["chosen_p"]
    # fp64 rule: divide, multiply root-to-leaf, add in insertion order
    d = [2.0 / 3.0, 1.0 / 3.0, (2.0 / 3.0) * (1.0 / 2.0), (2.0 / 3.0) * (1.0 / 2.0)]
    s = 0.0
    for x in d:
        s = s + x
    assert r["score"][0] == s
    assert abs(Fraction(r["score"][0]) - Fraction(*e["score_fraction"])) < Fraction(1, 10**12)
    c = o.candidate(-1, g["context"], 2, 4)
    for got, fr in zip(c[2], e["d_fractions"]):
        assert abs(Fraction(got) - Fraction(*fr)) < Fraction(1, 10**15)


@pytest.mark.parametrize("seed", range(6))
def test_match_is_substring_occurrence(oracle_mod, seed):
    rng = np.random.default_rng(seed)
    D = 5
    seqs = [rng.integers(0, 3, size=int(rng.integers(3, 15))).tolist() for _ in range(3)]
    o = _mk(oracle_mod, D, seqs)
    ctx = rng.integers(0, 3, size=9).tolist()
    matched = []
    for p in range(1, 9):
        c = o.candidate(-1, ctx, p, 4)
        expect = p <= D and occurrences(seqs, ctx[len(ctx) - p:]) > 0
        assert (c is not None) == expect
        matched.append(c is not None)
    # matched lengths form a prefix 1..p* (substring closure)
    assert matched == sorted(matched, reverse=True)
    assert o.candidate(-1, ctx, len(ctx) + 1, 4) is None          # p > t


@pytest.mark.parametrize("seed", range(12))
@pytest.mark.parametrize("linear", [False, True])
def test_expand_equals_bruteforce_greedy_bit_exact(oracle_mod, seed, linear):
    rng = np.random.default_rng(100 + seed)
    D = int(rng.integers(3, 7))
    seqs = [rng.integers(0, 3, size=int(rng.integers(4, 20))).tolist() for _ in range(4)]
    o = _mk(oracle_mod, D, seqs)
    ctx = seqs[0][: int(rng.integers(2, len(seqs[0]) + 1))]
    for p in range(1, min(len(ctx), D) + 1):
        for budget in (1, 2, 5, 40):
            want = greedy_tree(seqs, ctx[len(ctx) - p:], D, budget, linear)
            got = o.candidate(-1, ctx, p, budget, linear)
            assert (want is None) == (got is None)
            if want is None:
                continue
            assert got[0].tolist() == want[0] and got[1].tolist() == want[1]
            assert got[2].tolist() == want[2]           # D values, 0 ulp
            assert got[3] == want[3]                    # SCORE, 0 ulp


@pytest.mark.parametrize("seed", range(10))
def test_greedy_is_the_exhaustive_optimum(oracle_mod, seed):
    """D is non-increasing along every path, so best-first growth returns the
    maximum-SCORE connected sub-tree of its size; checked by enumeration on
    sub-trees with at most 12 candidate nodes, in exact rationals."""
    rng = np.random.default_rng(200 + seed)
    D = 4
    seqs = [rng.integers(0, 2, size=int(rng.integers(4, 9))).tolist() for _ in range(3)]
    o = _mk(oracle_mod, D, seqs)
    checked = 0
    for s in seqs:
        for p in (1, 2, 3):
            pat = s[:p]
            nodes = subtree_nodes(seqs, pat, D)
            if not (1 <= len(nodes) <= 12):
                continue
            for k in (1, 2, 3, 5, 12):
                got = o.candidate(-1, pat, p, k)
                assert len(got[0]) == min(k, len(nodes))
                exact = best_connected_score(nodes, k)
                assert abs(Fraction(got[3]) - exact) < Fraction(1, 10**12)
                checked += 1
    assert checked > 0


def test_single_child_chain_scores_its_length(oracle_mod):
    o = _mk(oracle_mod, 8, [[1, 2, 3, 4, 5, 6, 7, 8, 9]])
    tok, par, d, score = o.candidate(-1, [1, 2], 2, 10)
    assert tok.tolist() == [3, 4, 5, 6, 7, 8]            # stops at depth D = 8
    assert par.tolist() == [-1, 0, 1, 2, 3, 4]
    assert (d == 1.0).all() and score == 6.0
    tok, _, _, score = o.candidate(-1, [1, 2], 2, 3)     # stops at the budget
    assert tok.tolist() == [3, 4, 5] and score == 3.0
    # count drops along a unary chain do not change C (denominator is the sibling sum)
    o2 = _mk(oracle_mod, 8, [[1, 2, 3, 4], [1, 2, 3], [1, 2]])
    tok, _, d, score = o2.candidate(-1, [1], 1, 5)
    assert tok.tolist() == [2, 3, 4] and (d == 1.0).all() and score == 3.0


def test_equal_children_are_ordered_by_token_then_parent(oracle_mod):
    k = 4
    seqs = [[9, 30 - j] for j in range(k)]               # node [9] has k children, COUNT 1 each
    o = _mk(oracle_mod, 4, seqs)
    tok, par, d, score = o.candidate(-1, [9], 1, 10)
    assert tok.tolist() == [27, 28, 29, 30] and (d == 1.0 / k).all() and (par == -1).all()
    # same token under two parents with equal D: the earlier-added parent goes first
    seqs = [[1, 2, 7], [1, 3, 7]]
    o = _mk(oracle_mod, 4, seqs)
    tok, par, d, _ = o.candidate(-1, [1], 1, 10)
    assert tok.tolist() == [2, 3, 7, 7] and par.tolist() == [-1, -1, 0, 1]
    assert d.tolist() == [0.5, 0.5, 0.5, 0.5]


def test_denominator_is_sibling_sum_not_parent_count(oracle_mod):
    # [1] occurs 3 times, once at a sequence end: children 2 (x1), 3 (x1) -> C = 1/2, not 1/3
    o = _mk(oracle_mod, 4, [[1, 2], [1, 3], [5, 1]])
    tok, _, d, _ = o.candidate(-1, [1], 1, 4)
    assert tok.tolist() == [2, 3] and d.tolist() == [0.5, 0.5]


def test_budget_follows_alpha_p_with_cap(oracle_mod):
    o = oracle_mod.SuffixOracle(4, 1)
    assert [o.budget(1.0, p, 32) for p in (1, 2, 16, 40)] == [1, 2, 16, 32]
    assert [o.budget(2.0, p, 64) for p in (1, 24, 32, 33)] == [2, 48, 64, 64]
    assert [o.budget(1.5, p, 64) for p in (1, 2, 3)] == [1, 3, 4]
    assert o.budget(0.25, 3, 64) == 0


def test_selection_ties_first_in_loop_order_wins(oracle_mod):
    # global and per-request trees both give the chain 3,4 for p = 1 and p = 2 (score 2.0 at
    # budget 2).  Strict '>' keeps the first: the global tree, and there the smallest p that
    # reaches the top score.
    o = _mk(oracle_mod, 8, [[1, 2, 3, 4]], n_slots=2)
    o.slot_append(0, [1, 2, 3, 4, 1, 2])
    r = o.speculate([0], 2, 1.0, 2)
    assert r["score"][0] == 2.0 and r["chosen_tree"][0] == 0 and r["chosen_p"][0] == 2
    assert r["tokens"][0, :2].tolist() == [3, 4]
    # per-request only: same draft from the request's own text
    r = o.speculate([0], 2, 1.0, 2, flags=2)
    assert r["chosen_tree"][0] == 1 and r["chosen_p"][0] == 2 and r["tokens"][0, :2].tolist() == [3, 4]
    # p = 1 alone has budget 1
    r = o.speculate([0], 1, 1.0, 2)
    assert r["score"][0] == 1.0 and r["chosen_p"][0] == 1 and r["n_draft"][0] == 1
    # equal scores across p: a budget cap of 1 makes p = 1 and p = 2 tie at 1.0 -> p = 1
    r = o.speculate([0], 2, 1.0, 1)
    assert r["score"][0] == 1.0 and r["chosen_tree"][0] == 0 and r["chosen_p"][0] == 1
    # nothing matches: no tree
    o.slot_append(1, [77])
    r = o.speculate([1], 4, 2.0, 8)
    assert r["n_draft"][0] == 0 and r["chosen_tree"][0] == -1 and r["chosen_p"][0] == 0 and r["score"][0] == 0.0
    assert (r["tokens"][0] == -1).all() and (r["mask"][0] == 0).all()


def test_prompt_lookup_special_case(oracle_mod):
    """Per-request tree only; the pattern occurred exactly once before: the
    draft is the literal text that followed it, cut by the budget and by D - p."""
    text = [10, 11, 12, 13, 14, 15, 16, 17, 18, 19, 50, 51, 11, 12]
    D = 6
    o = oracle_mod.SuffixOracle(D, 1)
    o.slot_append(0, text)
    # p = 2 -> budget 16 but only D - p = 4 levels remain
    tok, par, d, score = o.candidate(0, text, 2, 16)
    assert tok.tolist() == [13, 14, 15, 16] and par.tolist() == [-1, 0, 1, 2] and score == 4.0
    # with a generous budget the shorter pattern reaches one level deeper and wins
    r = o.speculate([0], 2, 8.0, 64, flags=2)
    assert r["chosen_p"][0] == 1 and r["tokens"][0, :5].tolist() == [13, 14, 15, 16, 17] and r["n_draft"][0] == 5
    r = o.speculate([0], 2, 1.0, 64, flags=2)
    assert r["chosen_p"][0] == 2 and r["tokens"][0, :2].tolist() == [13, 14] and r["n_draft"][0] == 2


@pytest.mark.parametrize("seed", range(5))
def test_emitted_arrays_invariants(oracle_mod, seed):
    rng = np.random.default_rng(300 + seed)
    D, M = 8, 40
    seqs = [rng.integers(0, 4, size=60).tolist() for _ in range(4)]
    o = _mk(oracle_mod, D, seqs, n_slots=3)
    for s in range(3):
        o.slot_append(s, rng.integers(0, 4, size=30).tolist())
    r = o.speculate([0, 1, 2], 6, 6.0, 36, M=M)
    assert r["mask"].shape == (3, M, 2)
    for i in range(3):
        n, t = int(r["n_draft"][i]), o.slot_len(i)
        assert 0 < n <= o.budget(6.0, int(r["chosen_p"][i]), 36)
        assert 0.0 < r["score"][i] <= n
        depth = []
        for j in range(n):
            par = int(r["parents"][i, j])
            assert -1 <= par < j
            depth.append(1 if par < 0 else depth[par] + 1)
            row = int(r["mask"][i, j, 0]) | (int(r["mask"][i, j, 1]) << 32)
            prow = 0 if par < 0 else int(r["mask"][i, par, 0]) | (int(r["mask"][i, par, 1]) << 32)
            assert row == prow | (1 << j)
            assert bin(row).count("1") == depth[j]
            assert r["positions"][i, j] == t + depth[j] - 1
        # every root-to-node token path is a real continuation of the matched pattern
        ctx = o.slot_text(i).tolist()
        pat = ctx[len(ctx) - int(r["chosen_p"][i]):]
        src = seqs if r["chosen_tree"][i] == 0 else [ctx]
        for j in range(n):
            path, a = [], j
            while a >= 0:
                path.append(int(r["tokens"][i, a])); a = int(r["parents"][i, a])
            assert occurrences(src, pat + path[::-1]) > 0
        assert (r["parents"][i, n:] == -1).all() and (r["positions"][i, n:] == -1).all()


def test_threads_do_not_change_results(oracle_mod):
    rng = np.random.default_rng(9)
    o = _mk(oracle_mod, 8, [rng.integers(0, 5, size=80).tolist() for _ in range(4)], n_slots=6)
    for s in range(6):
        o.slot_append(s, rng.integers(0, 5, size=40).tolist())
    a = o.speculate(list(range(6)), 6, 2.0, 12, n_threads=1)
    b = o.speculate(list(range(6)), 6, 2.0, 12, n_threads=4)
    for k in a:
        assert np.array_equal(a[k], b[k])
    assert (a["visited"] > 0).all()


def test_per_request_budget_override(oracle_mod):
    o = _mk(oracle_mod, 8, [[1, 2, 3, 4, 5, 6]], n_slots=2)
    o.slot_append(0, [1, 2]); o.slot_append(1, [1, 2])
    r = o.speculate([0, 1], 2, 4.0, 8, budget_override=[1, -1])
    assert r["n_draft"].tolist() == [1, 4]


@pytest.mark.parametrize("seed", range(8))
def test_visit_counters_equal_bruteforce(oracle_mod, seed):
    """The work counters (the numerator of the benchmark's bytes, nodes-visited and candidate-trees
    figures).  descents: for every tree and pattern length, the tokens of the pattern that the walk
    finds before it stops = the longest prefix of the pattern that occurs; adds: draft nodes of
    every tree that was expanded, whether or not it is chosen; candidate trees: the expanded trees
    that got at least one draft node.  All from list scans, no trie."""
    rng = np.random.default_rng(500 + seed)
    D = int(rng.integers(2, 7))
    vocab = int(rng.integers(2, 5))
    seqs = [rng.integers(0, vocab, size=int(rng.integers(3, 25))).tolist() for _ in range(4)]
    o = _mk(oracle_mod, D, seqs, n_slots=3)
    texts = [rng.integers(0, vocab, size=int(rng.integers(1, 20))).tolist() for _ in range(3)]
    for s in range(3):
        o.slot_append(s, texts[s])
    for (P, alpha, cap, flags) in [(4, 2.0, 8, 0), (7, 1.0, 3, 0), (3, 4.0, 64, 4), (5, 1.5, 6, 1), (5, 1.5, 6, 2)]:
        r = o.speculate([0, 1, 2], P, alpha, cap, flags=flags)
        for s in range(3):
            ctx = texts[s]
            descents = adds = trees = 0
            for tree, src in ((0, seqs), (1, [ctx])):
                if (tree == 0 and flags & 2) or (tree == 1 and flags & 1):
                    continue
                for p in range(1, min(P, len(ctx), D) + 1):
                    pat = ctx[len(ctx) - p:]
                    k = 0
                    while k < p and occurrences(src, pat[:k + 1]) > 0:
                        k += 1
                    descents += k
                    if k == p:
                        size = len(greedy_tree(src, pat, D, o.budget(alpha, p, cap), bool(flags & 4))[0])
                        adds += size
                        trees += 1 if size else 0
            assert r["visited"][s].tolist() == [descents, adds, trees], (s, P, alpha, cap, flags)


def test_score_threshold_is_strict(oracle_mod):
    """Section 3.2: the draft is used only if SCORE > tau.  The hand-worked example scores
    2/3 + 1/3 + 1/3 + 1/3 (in that order, in binary64)."""
    g = json.load(open(os.path.join(GOLDEN, "hand_example.json")))
    o = _mk(oracle_mod, g["depth_cap"], g["global_sequences"])
    o.slot_append(0, g["context"])
    s = 0.0
    for x in (2.0 / 3.0, 1.0 / 3.0, (2.0 / 3.0) * (1.0 / 2.0), (2.0 / 3.0) * (1.0 / 2.0)):
        s = s + x
    below = np.nextafter(s, 0.0)
    for tau, kept in ((0.0, True), (1.0, True), (below, True), (s, False), (np.nextafter(s, 2.0), False), (5.0, False)):
        r = o.speculate([0], g["P"], g["alpha"], g["max_spec"], tau=float(tau))
        if kept:
            assert r["n_draft"][0] == 4 and r["score"][0] == s and r["chosen_tree"][0] == 0 and r["chosen_p"][0] == 2
        else:
            assert r["n_draft"][0] == 0 and r["score"][0] == 0.0 and r["chosen_tree"][0] == -1 and r["chosen_p"][0] == 0
            assert (r["tokens"][0] == -1).all() and (r["mask"][0] == 0).all()
    # the work counters do not depend on the threshold: every tree is still built
    a = o.speculate([0], g["P"], g["alpha"], g["max_spec"], tau=0.0)["visited"]
    b = o.speculate([0], g["P"], g["alpha"], g["max_spec"], tau=5.0)["visited"]
    assert np.array_equal(a, b)


def test_update_counter_is_min_depth_cap_context_length(oracle_mod):
    """Appending the token at context length t raises one COUNT per string that ends there:
    min(D, t) nodes (closed form of the online update of Section 3)."""
    o = oracle_mod.SuffixOracle(5, 2)
    o.slot_append(0, [1, 2, 3])
    assert o.slot_updates(0) == 1 + 2 + 3
    o.slot_append(0, [4, 5, 6, 7])
    assert o.slot_updates(0) == 1 + 2 + 3 + 4 + 5 + 5 + 5
    assert o.slot_updates(1) == 0
    o.slot_reset(0)
    assert o.slot_updates(0) == 0
