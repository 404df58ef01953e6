"""Helpers shared by the GPU parity tests: feed the same seeded inputs to the
CPU oracle and to the CUDA library (through its C ABI binding) and compare."""
import numpy as np
import torch

import oracle as oracle_pkg
import paper_2411_04975_b200 as sfx

DEV = "cuda:0"


def dev_i32(a):
    return torch.as_tensor(np.ascontiguousarray(a, dtype=np.int32), device=DEV)


def ragged(seqs):
    off = np.zeros(len(seqs) + 1, dtype=np.int64)
    if len(seqs):
        off[1:] = np.cumsum([len(s) for s in seqs])
    flat = (np.concatenate([np.asarray(s, dtype=np.int32) for s in seqs]) if len(seqs) and off[-1] > 0
            else np.zeros(0, dtype=np.int32))
    return off, flat.astype(np.int32)


def path_hashes(parent, token, depth):
    """A 64-bit hash of every node's root-to-node token path, from records in which a parent
    precedes its children (level by level: vectorised)."""
    n = len(token)
    h = np.zeros(n, dtype=np.uint64)
    K1, K2 = np.uint64(0x9E3779B97F4A7C15), np.uint64(0xC2B2AE3D27D4EB4F)
    with np.errstate(over="ignore"):
        for d in range(1, int(depth.max(initial=0)) + 1):
            idx = np.nonzero(depth == d)[0]
            hp = np.where(parent[idx] >= 0, h[np.maximum(parent[idx], 0)], np.uint64(0x1234567))
            x = (hp ^ (token[idx].astype(np.uint64) + np.uint64(1))) * K1
            x ^= x >> np.uint64(29)
            x *= K2
            x ^= x >> np.uint64(32)
            h[idx] = x
    return h


def canonical_nodes(parent, token, count, depth):
    """The tree as a sorted table (path hash, depth, count): equal tables = equal trees."""
    h = path_hashes(np.asarray(parent), np.asarray(token), np.asarray(depth))
    t = np.stack([h, np.asarray(depth).astype(np.uint64), np.asarray(count).astype(np.uint64)], axis=1)
    return t[np.lexsort((t[:, 2], t[:, 1], t[:, 0]))]


class Pair:
    """An oracle and a GPU store holding the same trees."""

    def __init__(self, corpus_seqs, *, vocab, D, n_slots, max_req_tokens, M=64, **kw):
        self.D, self.M, self.n_slots = D, M, n_slots
        self.o = oracle_pkg.SuffixOracle(D, n_slots)
        for s in corpus_seqs:
            self.o.global_insert(s)
        off, flat = ragged(corpus_seqs)
        if len(corpus_seqs):
            self.g = sfx.SuffixStore(dev_i32(flat) if flat.size else torch.zeros(0, dtype=torch.int32, device=DEV),
                                     torch.as_tensor(off, device=DEV), vocab=vocab, depth_cap=D,
                                     max_requests=n_slots, max_req_tokens=max_req_tokens, max_spec_cap=M, **kw)
        else:
            torch.cuda.set_device(0)
            self.g = sfx.SuffixStore(None, None, vocab=vocab, depth_cap=D, max_requests=n_slots,
                                     max_req_tokens=max_req_tokens, max_spec_cap=M, **kw)

    def close(self):
        self.g.free()
        self.o.close()

    def append(self, slots, token_lists, reset=None, oracle_threads=4):
        """slots: list of slot ids, -1 = global insert."""
        off, flat = ragged(token_lists)
        r = None if reset is None else torch.as_tensor(np.asarray(reset, dtype=np.uint8), device=DEV)
        self.g.append(dev_i32(slots), torch.as_tensor(off, device=DEV),
                      dev_i32(flat) if flat.size else torch.zeros(0, dtype=torch.int32, device=DEV), r)
        for i, s in enumerate(slots):
            if s < 0:
                self.o.global_insert(token_lists[i])
            elif reset is not None and reset[i]:
                self.o.slot_reset(s)
        idx = [i for i, s in enumerate(slots) if s >= 0]
        self.o.slot_append_batch([slots[i] for i in idx], [token_lists[i] for i in idx], n_threads=oracle_threads)

    def check_tree(self, tree):
        """The GPU tree, enumerated on the device, has exactly the oracle's nodes with the oracle's
        counts; and every path of the oracle's tree, looked up on the GPU, has the same COUNT."""
        depth, parent, tok, cnt = self.o.dump(tree)
        n = len(tok)
        if tree < 0:
            assert self.g.stats()["global_nodes"] == n
        else:
            info = self.g.slot_info(dev_i32([tree]))
            assert int(info["nodes"][0]) == n
            assert int(info["len"][0]) == self.o.slot_len(tree)
        # the GPU tree enumerated on the device, node by node: the same set of (path, depth, count)
        rec = {k: v.cpu().numpy() for k, v in self.g.enumerate(tree, n + 8).items()}
        assert len(rec["token"]) == n
        if n:
            assert (rec["parent"] < np.arange(n)).all()
            assert np.array_equal(canonical_nodes(rec["parent"], rec["token"], rec["count"], rec["depth"]),
                                  canonical_nodes(parent, tok, cnt, depth)), f"tree {tree}: node sets differ"
        if n == 0:
            return
        off = np.zeros(n + 1, dtype=np.int64)
        off[1:] = np.cumsum(depth)
        flat = np.empty(int(off[-1]), dtype=np.int32)
        # pre-order: a node's path is its parent's path plus its token
        for i in range(n):
            b = off[i]
            if parent[i] >= 0:
                pb = off[parent[i]]
                flat[b:b + depth[i] - 1] = flat[pb:pb + depth[i] - 1]
            flat[b + depth[i] - 1] = tok[i]
        got = self.g.query_counts(dev_i32(np.full(n, tree)), torch.as_tensor(off, device=DEV), dev_i32(flat))
        got = got.cpu().numpy()
        bad = np.nonzero(got != cnt)[0]
        assert bad.size == 0, f"tree {tree}: {bad.size} of {n} counts differ, first path " \
                              f"{flat[off[bad[0]]:off[bad[0] + 1]].tolist()} gpu {got[bad[0]]} oracle {cnt[bad[0]]}"

    def speculate_both(self, slots, P, alpha, max_spec, flags=0, budget_cap=None, oracle_threads=4, tau=0.0):
        bc = None if budget_cap is None else dev_i32(budget_cap)
        out = self.g.speculate(dev_i32(slots), P, alpha, max_spec, flags, bc, tau=tau)
        torch.cuda.synchronize()
        got = {k: v.cpu().numpy() for k, v in out.items()}
        got["mask"] = got["mask"].view(np.uint32)
        want = self.o.speculate(slots, P, alpha, max_spec, M=self.M, flags=flags, budget_override=budget_cap,
                                n_threads=oracle_threads, tau=tau)
        return got, want

    def check_speculate(self, slots, P, alpha, max_spec, flags=0, budget_cap=None, tau=0.0):
        got, want = self.speculate_both(slots, P, alpha, max_spec, flags, budget_cap, tau=tau)
        assert_same_drafts(got, want)
        return got, want


def assert_same_drafts(got, want):
    """Bit-exact: integer arrays equal, fp64 scores equal as bit patterns."""
    for k in ("n_draft", "chosen_tree", "chosen_p", "tokens", "parents", "positions", "mask"):
        if not np.array_equal(got[k], want[k]):
            bad = np.nonzero((got[k] != want[k]).reshape(len(got[k]), -1).any(axis=1))[0]
            i = int(bad[0])
            raise AssertionError(
                f"{k} differs for {bad.size} requests; first request {i}: gpu n={got['n_draft'][i]} "
                f"tree={got['chosen_tree'][i]} p={got['chosen_p'][i]} score={got['score'][i]!r} tokens="
                f"{got['tokens'][i][:8].tolist()} | oracle n={want['n_draft'][i]} tree={want['chosen_tree'][i]} "
                f"p={want['chosen_p'][i]} score={want['score'][i]!r} tokens={want['tokens'][i][:8].tolist()}")
    assert np.array_equal(got["score"].view(np.int64), want["score"].view(np.int64)), "score bits differ"
