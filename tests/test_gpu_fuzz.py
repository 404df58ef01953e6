"""Randomised differential test: small stores with random shapes, vocabularies, depth caps and
call sequences (batched prompt build or appends, one-launch steps or append + speculate, global
inserts in between, flags, budget caps and score thresholds), every draft compared bit by bit with the oracle and
the trees compared node by node at the end."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def U():
    import gpu_util
    return gpu_util


def _seqs(rng, n, lo, hi, vocab, zipf):
    out = []
    for _ in range(n):
        L = int(rng.integers(lo, hi + 1))
        s = np.minimum(rng.zipf(1.3, size=L) - 1, vocab - 1) if zipf else rng.integers(0, vocab, size=L)
        if rng.random() < 0.3 and L > 4:                         # a periodic stretch
            per = int(rng.integers(1, 4))
            a = int(rng.integers(0, L - 2))
            b = int(rng.integers(a + 1, L))
            s[a:b] = np.resize(rng.integers(0, vocab, size=per), b - a)
        out.append(s.astype(np.int32))
    return out


def _empty():
    return torch.zeros(0, dtype=torch.int32, device="cuda:0")


def _scenario(U, seed):
    rng = np.random.default_rng(seed)
    vocab = int(rng.choice([2, 3, 5, 17, 60, 300, 5000]))
    D = int(rng.choice([1, 2, 3, 5, 8, 13, 16, 24, 32]))
    zipf = bool(rng.random() < 0.5)
    n_slots = int(rng.choice([1, 3, 8, 20, 40, 150, 310]))
    maxtok = int(rng.choice([40, 200, 700]))
    corpus = _seqs(rng, int(rng.choice([0, 1, 5, 30])), 1, int(rng.choice([5, 60, 400, 2000])), vocab, zipf)
    pr = U.Pair(corpus, vocab=vocab, D=D, n_slots=n_slots, max_req_tokens=maxtok + 64)
    slots = list(range(n_slots))
    prompts = _seqs(rng, n_slots, 0, maxtok // 2, vocab, zipf)
    if rng.random() < 0.5:
        off, flat = U.ragged(prompts)
        pr.g.build_requests(np.asarray(slots, dtype=np.int32), off, U.dev_i32(flat) if flat.size else _empty())
        for s in slots:
            pr.o.slot_reset(s)
        pr.o.slot_append_batch(slots, prompts, n_threads=4)
    else:
        pr.append(slots, prompts, reset=[1] * n_slots)
    for _ in range(int(rng.integers(2, 6))):
        P = int(rng.integers(1, 33))
        alpha = float(rng.choice([0.5, 1.0, 1.5, 2.0, 4.0]))
        max_spec = int(rng.integers(1, 65))
        flags = int(rng.choice([0, 0, 0, 1, 2, 4, 5, 6]))
        sub = slots if rng.random() < 0.7 else sorted(rng.choice(n_slots, size=max(1, n_slots // 2), replace=False).tolist())
        cap = rng.integers(-1, 40, size=len(sub)).astype(np.int32) if rng.random() < 0.3 else None
        tau = float(rng.choice([0.0, 0.0, 0.25, 1.0, 1.5, 3.0, 8.0]))   # score threshold of Section 3.2
        lists = _seqs(rng, len(sub), 0, int(rng.choice([1, 4, 12])), vocab, zipf)
        lists = [l[:max(0, maxtok + 60 - pr.o.slot_len(s))] for l, s in zip(lists, sub)]   # stay inside the text buffer
        if rng.random() < 0.5:
            off, flat = U.ragged(lists)
            out = pr.g.step(U.dev_i32(sub), torch.as_tensor(off, device=U.DEV), U.dev_i32(flat) if flat.size else _empty(),
                            P, alpha, max_spec, flags, None if cap is None else U.dev_i32(cap), tau=tau)
            torch.cuda.synchronize()
            pr.o.slot_append_batch(sub, lists, n_threads=4)
            want = pr.o.speculate(sub, P, alpha, max_spec, M=64, flags=flags, budget_override=cap, n_threads=4, tau=tau)
            got = {k: v.cpu().numpy() for k, v in out.items()}
            got["mask"] = got["mask"].view(np.uint32)
            U.assert_same_drafts(got, want)
        else:
            pr.append(sub, lists)
            pr.check_speculate(sub, P, alpha, max_spec, flags, cap, tau=tau)
        if rng.random() < 0.4:
            finished = _seqs(rng, int(rng.integers(1, 4)), 1, 120, vocab, zipf)
            pr.append([-1] * len(finished), finished)
    pr.check_tree(-1)
    for s in rng.choice(n_slots, size=min(3, n_slots), replace=False).tolist():
        pr.check_tree(int(s))
    pr.close()


@pytest.mark.parametrize("block", range(4))
def test_random_scenarios(U, block):
    for k in range(40):
        seed = 900000 + block * 1000 + k
        try:
            _scenario(U, seed)
        except AssertionError as e:
            raise AssertionError(f"scenario seed {seed}: {e}") from e
