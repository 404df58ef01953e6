"""Brute-force definitions used to pin the CPU oracle.

Nothing here builds a trie: counts come from scanning the sequences, children
come from scanning for one-token extensions, and the best tree comes from a
plain arg-max over a list or from exhaustive enumeration.  Python floats are
IEEE doubles with correctly rounded / and *, and Python never fuses them, so
the fp64 values computed here are bit-comparable with the oracle's.
"""
from fractions import Fraction
from itertools import combinations


def occurrences(seqs, path):
    """Number of (sequence, position) occurrences of `path` (COUNT below Eq. 2)."""
    path = list(path)
    n = len(path)
    c = 0
    for s in seqs:
        s = list(s)
        for i in range(len(s) - n + 1):
            if s[i:i + n] == path:
                c += 1
    return c


def distinct_substrings(seqs, D):
    out = set()
    for s in seqs:
        s = list(s)
        for i in range(len(s)):
            for l in range(1, min(D, len(s) - i) + 1):
                out.add(tuple(s[i:i + l]))
    return out


def children(seqs, path, D):
    """{token: count} of the one-token extensions of `path` (empty at depth D)."""
    path = list(path)
    if len(path) >= D:
        return {}
    out = {}
    for s in seqs:
        s = list(s)
        n = len(path)
        for i in range(len(s) - n):
            if s[i:i + n] == path:
                out[s[i + n]] = out.get(s[i + n], 0) + 1
    return out


def greedy_tree(seqs, pattern, D, budget, linear=False):
    """Algorithm 1's ExpandSpeculationTree by list scans.  Returns (tokens,
    parents, dvals, score) or None when the pattern does not occur."""
    pattern = list(pattern)
    if len(pattern) > D or occurrences(seqs, pattern) == 0:
        return None
    tokens, parents, dvals, paths = [], [], [], []
    cand = []  # (d, token, parent_index, path)

    def push(path, d_parent, parent_index):
        ch = children(seqs, path, D)
        tot = sum(ch.values())
        for tok, cnt in ch.items():
            cand.append((d_parent * (float(cnt) / float(tot)), tok, parent_index, path + [tok]))

    push(pattern, 1.0, -1)
    score = 0.0
    while len(tokens) < budget and cand:
        best = 0
        for i in range(1, len(cand)):
            a, b = cand[i], cand[best]
            if a[0] > b[0] or (a[0] == b[0] and (a[1] < b[1] or (a[1] == b[1] and a[2] < b[2]))):
                best = i
        d, tok, par, path = cand.pop(best)
        idx = len(tokens)
        tokens.append(tok); parents.append(par); dvals.append(d); paths.append(path)
        score = score + d
        if linear:
            cand.clear()
        push(path, d, idx)
    return tokens, parents, dvals, score


def subtree_nodes(seqs, pattern, D):
    """All nodes strictly below the pattern's node: list of (path, parent_pos, exact D)."""
    nodes = []

    def rec(path, d_parent, parent_pos):
        ch = children(seqs, path, D)
        tot = sum(ch.values())
        for tok in sorted(ch):
            d = d_parent * Fraction(ch[tok], tot)
            nodes.append((path + [tok], parent_pos, d))
            rec(path + [tok], d, len(nodes) - 1)

    rec(list(pattern), Fraction(1), -1)
    return nodes


def best_connected_score(nodes, k):
    """Max over connected sub-trees (containing the root N_p) with exactly
    min(k, len(nodes)) draft nodes of the exact sum of D."""
    k = min(k, len(nodes))
    best = Fraction(0)
    for comb in combinations(range(len(nodes)), k):
        chosen = set(comb)
        if all(nodes[i][1] == -1 or nodes[i][1] in chosen for i in comb):
            s = sum((nodes[i][2] for i in comb), Fraction(0))
            if s > best:
                best = s
    return best
