"""GPU parity: the CUDA path against the CPU oracle, element by element, on the
same seeded inputs, through the C ABI."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def U():
    import gpu_util
    return gpu_util


def _rand_seqs(rng, n, lo, hi, vocab):
    return [rng.integers(0, vocab, size=int(rng.integers(lo, hi + 1))).astype(np.int32) for _ in range(n)]


# ---------------------------------------------------------------- offline build (a1)
@pytest.mark.parametrize("D", [1, 2, 3, 5, 8, 13, 32])
@pytest.mark.parametrize("vocab", [2, 50])
def test_build_counts_match_oracle(U, D, vocab):
    rng = np.random.default_rng(D * 100 + vocab)
    seqs = _rand_seqs(rng, 12, 0, 300, vocab) + [np.full(70, 1, dtype=np.int32)]
    pr = U.Pair(seqs, vocab=vocab, D=D, n_slots=1, max_req_tokens=8)
    pr.check_tree(-1)
    # absent and over-long paths count 0
    paths = [[vocab - 1] * (D + 1), [0] * min(D, 3) + [vocab - 1] * 0]
    off, flat = U.ragged(paths)
    got = pr.g.query_counts(U.dev_i32([-1, -1]), torch.as_tensor(off, device=U.DEV), U.dev_i32(flat)).cpu().numpy()
    assert got[0] == 0 and got[1] == pr.o.count(-1, paths[1])
    pr.close()


def test_build_spans_many_tiles_and_ragged_tail(U):
    # > 2048-element sort/scan tiles, ragged last tile, repeated spans
    from workload.generator import get_workload
    w = get_workload("tiny")
    corpus = w.corpus()
    seqs = [corpus[i * 512:(i + 1) * 512] for i in range(64)]
    seqs[-1] = seqs[-1][:301]
    pr = U.Pair(seqs, vocab=32000, D=32, n_slots=1, max_req_tokens=8)
    pr.check_tree(-1)
    pr.close()


def test_build_empty_corpus_and_bad_inputs(U):
    import paper_2411_04975_b200 as sfx
    pr = U.Pair([], vocab=10, D=4, n_slots=2, max_req_tokens=16)
    assert pr.g.stats()["global_nodes"] == 0
    got, _ = pr.check_speculate([0, 1], 4, 2.0, 8)
    assert (got["n_draft"] == 0).all()
    pr.close()
    with pytest.raises(sfx.SuffixSpecError):       # token outside [0, V)
        U.Pair([np.array([1, 2, 99], dtype=np.int32)], vocab=10, D=4, n_slots=1, max_req_tokens=8)
    with pytest.raises(sfx.SuffixSpecError):       # depth cap beyond the limit
        U.Pair([np.array([1, 2], dtype=np.int32)], vocab=10, D=33, n_slots=1, max_req_tokens=8)
    with pytest.raises(sfx.SuffixSpecError):
        U.Pair([np.array([1, 2], dtype=np.int32)], vocab=10, D=4, n_slots=1, max_req_tokens=8, M=65)


# ---------------------------------------------------------------- online update (a2, a3, a4)
@pytest.mark.parametrize("D", [1, 4, 32])
@pytest.mark.parametrize("vocab", [1, 2, 40])
def test_append_matches_oracle_after_every_batch(U, D, vocab):
    rng = np.random.default_rng(7 * D + vocab)
    n_slots = 5
    pr = U.Pair(_rand_seqs(rng, 3, 5, 40, vocab), vocab=vocab, D=D, n_slots=n_slots, max_req_tokens=400)
    # prompts (reset), one slot left empty
    slots = [0, 1, 2, 3]
    pr.append(slots, _rand_seqs(rng, 4, 0, 120, vocab), reset=[1, 1, 1, 1])
    for s in range(n_slots):
        pr.check_tree(s)
    for step in range(6):
        k = int(rng.integers(1, n_slots + 1))
        slots = sorted(rng.choice(n_slots, size=k, replace=False).tolist())
        toks = _rand_seqs(rng, k, 0, 9, vocab)
        if step == 3:                               # long runs of one token (periodic tail)
            toks = [np.full(40, vocab - 1, dtype=np.int32) for _ in slots]
        pr.append(slots, toks)
        for s in range(n_slots):
            pr.check_tree(s)
    # a new request reuses a slot
    pr.append([1, 4], _rand_seqs(rng, 2, 30, 60, vocab), reset=[1, 0])
    for s in (1, 4):
        pr.check_tree(s)
    pr.check_tree(-1)                               # the global tree was never touched
    pr.close()


@pytest.mark.parametrize("vocab", [2, 30])
def test_global_online_insert(U, vocab):
    rng = np.random.default_rng(vocab)
    pr = U.Pair(_rand_seqs(rng, 6, 10, 200, vocab), vocab=vocab, D=8, n_slots=2, max_req_tokens=64)
    for step in range(4):
        seqs = _rand_seqs(rng, 3, 0, 90, vocab)
        pr.append([-1, 0, -1, -1], [seqs[0], rng.integers(0, vocab, size=5).astype(np.int32), seqs[1], seqs[2]])
        pr.check_tree(-1)
        pr.check_tree(0)
    assert pr.g.stats()["global_tokens"] == pr.o.count(-1, [0]) + sum(
        pr.o.count(-1, [v]) for v in range(1, vocab))
    pr.close()
    # into an empty global tree
    pr = U.Pair([], vocab=vocab, D=5, n_slots=1, max_req_tokens=8)
    pr.append([-1, -1], _rand_seqs(rng, 2, 20, 50, vocab))
    pr.check_tree(-1)
    pr.close()


@pytest.mark.parametrize("vocab,D,zipf", [(2, 32, False), (3, 7, False), (40, 32, True), (5000, 32, True),
                                          (5000, 16, False)])
def test_global_insert_many_paths_and_items(U, vocab, D, zipf):
    """Global inserts larger than one pass of the insert kernel (more than 1,024 start positions, more
    than 256 items in one call), mixed with request items, on trees where many paths share their
    parents (tiny vocabularies, periodic text) and on trees with long child runs."""
    rng = np.random.default_rng(1000 * vocab + D)

    def seqs(n, lo, hi):
        out = []
        for _ in range(n):
            L = int(rng.integers(lo, hi + 1))
            s = np.minimum(rng.zipf(1.2, size=L) - 1, vocab - 1) if zipf else rng.integers(0, vocab, size=L)
            if L > 8 and rng.random() < 0.5:                      # a copy of an earlier stretch, and a periodic one
                a, b = sorted(rng.integers(0, L, size=2).tolist())
                s[b:] = np.resize(s[a:b + 1], L - b)
            out.append(s.astype(np.int32))
        return out

    pr = U.Pair(seqs(20, 50, 600), vocab=vocab, D=D, n_slots=4, max_req_tokens=256)
    # one long sequence and a few short ones: several passes, paths that end early
    pr.append([-1, -1, 2, -1], [seqs(1, 2500, 2500)[0], seqs(1, 1, 1)[0], seqs(1, 30, 30)[0], seqs(1, 700, 700)[0]])
    pr.check_tree(-1)
    pr.check_tree(2)
    # more items than one round of the item scan takes, empty sequences among them
    many = seqs(600, 0, 9)
    slots = [-1] * len(many)
    slots[100], slots[400] = 0, 1
    pr.append(slots, many)
    pr.check_tree(-1)
    pr.check_tree(0)
    # the same text again: every node exists, only counts change
    pr.append([-1] * 3, [np.concatenate(many[:300]), np.concatenate(many[300:]), many[7]])
    pr.check_tree(-1)
    assert pr.g.stats()["global_status"] == 0
    pr.check_speculate([0, 1, 2], 8, 2.0, 16)
    pr.close()


def test_global_insert_bad_token_and_full_pool(U):
    rng = np.random.default_rng(77)
    vocab, D = 50, 8
    base = [rng.integers(0, vocab, size=80).astype(np.int32) for _ in range(3)]
    # a token outside the vocabulary ends its sequence there; the other sequences are not affected
    pr = U.Pair(base, vocab=vocab, D=D, n_slots=1, max_req_tokens=16)
    good = rng.integers(0, vocab, size=300).astype(np.int32)
    bad = good.copy()
    bad[120] = vocab
    other = rng.integers(0, vocab, size=1500).astype(np.int32)
    off, flat = U.ragged([bad, other])
    pr.g.append(U.dev_i32([-1, -1]), torch.as_tensor(off, device=U.DEV), U.dev_i32(flat))
    pr.o.global_insert(bad[:120]); pr.o.global_insert(other)
    pr.check_tree(-1)
    assert pr.g.stats()["global_status"] == 8
    pr.close()
    # a pool without room: the status bit is set, the store stays usable and every count that is
    # there is at most the oracle's
    pr = U.Pair(base, vocab=vocab, D=D, n_slots=1, max_req_tokens=16, global_extra_nodes=500)
    off, flat = U.ragged([other])
    pr.g.append(U.dev_i32([-1]), torch.as_tensor(off, device=U.DEV), U.dev_i32(flat))
    st = pr.g.stats()
    assert st["global_status"] & 4 and st["global_pool_used"] <= st["global_pool_cap"]
    pr.o.global_insert(other)
    depth, parent, tok, cnt = pr.o.dump(-1)
    sel = np.nonzero(depth <= 2)[0]
    paths = [[int(tok[i])] if depth[i] == 1 else [int(tok[parent[i]]), int(tok[i])] for i in sel]
    qoff, qflat = U.ragged(paths)
    got = pr.g.query_counts(U.dev_i32(np.full(len(paths), -1)), torch.as_tensor(qoff, device=U.DEV), U.dev_i32(qflat))
    assert (got.cpu().numpy() <= cnt[sel]).all()
    # later inserts are refused as a whole, speculation still works
    before = pr.g.stats()["global_tokens"]
    pr.g.append(U.dev_i32([-1]), torch.as_tensor(off, device=U.DEV), U.dev_i32(flat))
    assert pr.g.stats()["global_tokens"] == before
    pr.g.append(U.dev_i32([0]), torch.as_tensor(np.array([0, 10]), device=U.DEV), U.dev_i32(other[:10]),
                torch.ones(1, dtype=torch.uint8, device=U.DEV))
    out = pr.g.speculate(U.dev_i32([0]), 4, 2.0, 8)
    torch.cuda.synchronize()
    assert int(out["n_draft"][0]) >= 0
    pr.close()


def test_pool_overflow_is_reported_and_tree_stays_consistent(U):
    rng = np.random.default_rng(3)
    pr = U.Pair([], vocab=1000, D=8, n_slots=2, max_req_tokens=64, slot_pool_nodes=100)
    toks = rng.integers(0, 1000, size=60).astype(np.int32)
    off, flat = U.ragged([toks, toks[:5]])
    pr.g.append(U.dev_i32([0, 1]), torch.as_tensor(off, device=U.DEV), U.dev_i32(flat))
    info = pr.g.slot_info(U.dev_i32([0, 1, 7]))
    status = info["status"].cpu().numpy()
    assert status[0] & 2 and status[1] == 0 and status[2] == 1
    kept = int(info["len"][0])
    assert 0 < kept < 60
    pr.o.slot_append(0, toks[:kept]); pr.o.slot_append(1, toks[:5])
    pr.check_tree(0); pr.check_tree(1)
    out = pr.g.speculate(U.dev_i32([0, 1]), 4, 2.0, 8)
    assert int(out["n_draft"][0]) == 0 and int(out["status"][0]) & 2
    # text buffer limit
    pr.g.append(U.dev_i32([1]), torch.as_tensor(np.array([0, 70]), device=U.DEV), U.dev_i32(np.arange(70) % 3))
    assert int(pr.g.slot_info(U.dev_i32([1]))["status"][0]) & 2
    # a token outside the vocabulary stops that slot only
    pr.g.append(U.dev_i32([0]), torch.as_tensor(np.array([0, 2]), device=U.DEV), U.dev_i32([5, 1000]),
                torch.ones(1, dtype=torch.uint8, device=U.DEV))
    assert int(pr.g.slot_info(U.dev_i32([0]))["status"][0]) == 8
    pr.close()


# ---------------------------------------------------------------- speculate (a5 - a8)
@pytest.mark.parametrize("seed", range(4))
def test_speculate_small_vocab_stress(U, seed):
    """Low-entropy text: wide child runs, many equal scores (tie rules), deep trees."""
    rng = np.random.default_rng(40 + seed)
    vocab = [2, 3, 6, 12][seed]
    D = [32, 8, 16, 5][seed]
    n_slots = 24
    pr = U.Pair(_rand_seqs(rng, 20, 50, 400, vocab), vocab=vocab, D=D, n_slots=n_slots, max_req_tokens=300)
    pr.append(list(range(n_slots)), _rand_seqs(rng, n_slots, 0, 200, vocab), reset=[1] * n_slots)
    slots = list(range(n_slots))
    for (P, alpha, ms) in [(8, 1.0, 8), (32, 2.0, 64), (40, 1.5, 33), (3, 0.5, 64), (16, 4.0, 64), (5, 8.0, 1)]:
        for flags in (0, 1, 2, 4, 5, 6):
            pr.check_speculate(slots, P, alpha, ms, flags)
    bc = rng.integers(-1, 20, size=n_slots).astype(np.int32)
    pr.check_speculate(slots, 16, 2.0, 64, 0, bc)
    # subset of the batch, in another order
    pr.check_speculate([5, 3, 17], 16, 2.0, 64)
    pr.close()


def test_speculate_tiny_config(U):
    """The tiny workload at full size."""
    from workload.generator import get_workload
    w = get_workload("tiny")
    c = w.cfg
    corpus = w.corpus()
    seqs = [corpus[i * c.seq_len:(i + 1) * c.seq_len] for i in range(c.n_seqs)]
    pr = U.Pair(seqs, vocab=c.vocab, D=c.depth_cap, n_slots=c.batch, max_req_tokens=c.prompt_len + 64, M=c.max_spec)
    pr.append(list(range(c.batch)), w.prompts(), reset=[1] * c.batch)
    got, want = pr.check_speculate(list(range(c.batch)), c.max_pattern, c.alpha, c.max_spec)
    assert (got["n_draft"] > 0).any()
    for s in range(c.batch):
        pr.check_tree(s)
    pr.close()


def test_speculate_wide_runs(U):
    """A match node with thousands of children (several 32-entry chunks, the
    32-way search) and a bounded frontier much smaller than the run."""
    rng = np.random.default_rng(5)
    vocab = 5000
    seqs = [np.stack([np.zeros(3000, dtype=np.int32), rng.integers(1, vocab, size=3000).astype(np.int32)],
                     axis=1).reshape(-1)]
    seqs += _rand_seqs(rng, 10, 100, 300, vocab)
    pr = U.Pair(seqs, vocab=vocab, D=6, n_slots=4, max_req_tokens=700)
    prompts = [np.concatenate([s[:600], [0]]).astype(np.int32) for s in (seqs[0], seqs[0][2:], seqs[1], seqs[2])]
    pr.append([0, 1, 2, 3], prompts, reset=[1] * 4)
    for (P, alpha, ms) in [(1, 64.0, 64), (4, 16.0, 64), (6, 2.0, 7)]:
        pr.check_speculate([0, 1, 2, 3], P, alpha, ms)
    for s in range(4):
        pr.check_tree(s)
    pr.check_tree(-1)
    pr.close()


def test_speculate_edge_cases(U):
    import paper_2411_04975_b200 as sfx
    rng = np.random.default_rng(1)
    pr = U.Pair(_rand_seqs(rng, 4, 20, 60, 4), vocab=4, D=8, n_slots=3, max_req_tokens=64, M=40)
    pr.append([0, 2], _rand_seqs(rng, 2, 10, 30, 4), reset=[1, 1])
    # slot 1 is empty (t = 0): no pattern, no draft
    got, _ = pr.check_speculate([0, 1, 2], 8, 2.0, 40)
    assert got["n_draft"][1] == 0 and got["chosen_tree"][1] == -1
    assert got["mask"].shape == (3, 40, 2)
    # max_spec 0 and alpha 0: empty drafts everywhere
    got, _ = pr.check_speculate([0, 2], 8, 2.0, 0)
    assert (got["n_draft"] == 0).all()
    got, _ = pr.check_speculate([0, 2], 8, 0.0, 40)
    assert (got["n_draft"] == 0).all()
    # out-of-range slot: status only
    out = pr.g.speculate(U.dev_i32([0, 9]), 8, 2.0, 40)
    assert int(out["status"][1]) == 1 and int(out["n_draft"][1]) == 0 and int(out["status"][0]) == 0
    # argument errors are return codes
    for bad in (dict(P=0), dict(max_spec=41), dict(flags=3), dict(alpha=float("nan"))):
        kw = dict(P=8, alpha=2.0, max_spec=40, flags=0)
        kw.update(bad)
        with pytest.raises(sfx.SuffixSpecError):
            pr.g.speculate(U.dev_i32([0]), kw["P"], kw["alpha"], kw["max_spec"], kw["flags"])
    with pytest.raises(sfx.SuffixSpecError):
        pr.g.speculate(U.dev_i32([0, 1, 2, 0]), 8, 2.0, 40)        # more requests than slots
    # n = 0 is a no-op
    pr.g.speculate(torch.zeros(0, dtype=torch.int32, device=U.DEV), 8, 2.0, 40)
    pr.g.append(torch.zeros(0, dtype=torch.int32, device=U.DEV), torch.zeros(1, dtype=torch.int64, device=U.DEV),
                torch.zeros(0, dtype=torch.int32, device=U.DEV))
    pr.close()


def test_speculate_is_deterministic(U):
    rng = np.random.default_rng(2)
    pr = U.Pair(_rand_seqs(rng, 10, 100, 300, 5), vocab=5, D=16, n_slots=16, max_req_tokens=256)
    pr.append(list(range(16)), _rand_seqs(rng, 16, 50, 200, 5), reset=[1] * 16)
    a = pr.g.speculate(U.dev_i32(list(range(16))), 16, 2.0, 64)
    a = {k: v.clone() for k, v in a.items()}
    b = pr.g.speculate(U.dev_i32(list(range(16))), 16, 2.0, 64)
    for k in a:
        if k != "packed":                                        # the one buffer behind the views: has padding
            assert torch.equal(a[k], b[k])
    pr.close()


# ---------------------------------------------------------------- the named workloads, scaled so the oracle takes seconds
def _config_pair(U, name, n_seqs, batch, prompt_len=None, extra_tokens=64):
    from workload.generator import get_workload
    kw = dict(n_seqs=n_seqs, batch=batch)
    if prompt_len:
        kw["prompt_len"] = prompt_len
    w = get_workload(name, **kw)
    c = w.cfg
    corpus = w.corpus()
    seqs = [corpus[i * c.seq_len:(i + 1) * c.seq_len] for i in range(c.n_seqs)]
    pr = U.Pair(seqs, vocab=c.vocab, D=c.depth_cap, n_slots=c.batch, max_req_tokens=c.prompt_len + extra_tokens,
                M=c.max_spec)
    return w, c, pr


@pytest.mark.parametrize("name,n_seqs,batch", [("agentic", 300, 6), ("large_batch", 256, 24),
                                               ("low_repetition", 256, 32)])
def test_configs_scaled_prompts_then_decode_steps(U, name, n_seqs, batch):
    """Corpus cut to a few hundred sequences, prompts at full length (8,192 / 4,096 tokens),
    every other parameter as the workload defines it; three decode steps of appends."""
    w, c, pr = _config_pair(U, name, n_seqs, batch)
    prompts = w.prompts()
    pr.append(list(range(batch)), prompts, reset=[1] * batch)
    pr.check_tree(-1)
    for s in (0, batch - 1):
        pr.check_tree(s)
    got, _ = pr.check_speculate(list(range(batch)), c.max_pattern, c.alpha, c.max_spec)
    assert (got["n_draft"] > 0).any()
    cont = [w.continuation(i, prompts[i], length=40) for i in range(batch)]
    cur = 0
    for step, k in enumerate((1, 7, 3)):
        pr.append(list(range(batch)), [x[cur:cur + k] for x in cont])
        cur += k
        pr.check_speculate(list(range(batch)), c.max_pattern, c.alpha, c.max_spec)
        pr.check_speculate(list(range(batch)), c.max_pattern, c.alpha, c.max_spec, flags=4)
    pr.check_tree(1)
    pr.close()


def test_closed_loop_scaled(U):
    """The closed-loop workload in miniature: speculate, accept against the hidden continuation, append
    accepted + bonus tokens, insert finished outputs into the global tree, refill the slot."""
    from workload.closed_loop import ClosedLoop
    w, c, pr = _config_pair(U, "closed_loop", 128, 12, prompt_len=300, extra_tokens=80)
    loop = ClosedLoop(w, 12, prompt_len=300, out_lo=10, out_hi=60)
    pr.append(*loop.start())
    for step in range(40):
        got, _ = pr.check_speculate(list(range(12)), c.max_pattern, c.alpha, c.max_spec)
        slots, lists, reset = loop.advance(got)
        pr.append(slots, lists, reset)
        if step % 13 == 0:
            pr.check_tree(-1)
            pr.check_tree(step % 12)
    s = loop.summary()
    assert s["finished_requests"] >= 12 and s["mean_accepted_drafts"] > 0.5
    pr.check_tree(-1)
    for sl in range(12):
        pr.check_tree(sl)
    pr.close()


@pytest.mark.parametrize("name,one_launch", [("large_batch", False), ("large_batch", True), ("agentic", True),
                                             ("low_repetition", True)])
def test_full_size_sampled_against_oracle(U, name, one_launch):
    """The named workloads at full size (large_batch: 4,194,304-token global tree, 256 requests x 4,096-token
    prompts; agentic: 64 requests x 8,192 tokens, P = 24; low_repetition: 512 requests) in the launch
    configurations bench.py times: sd_append + sd_speculate, and (one_launch) prompts through
    sd_build_requests and every decode step as one sd_step.  The oracle holds the full global tree
    but only a sample of the requests; their rows must be bit-exact, and every row must satisfy the
    properties that hold for any draft."""
    from workload.generator import accept_schedule, get_workload
    import oracle as oracle_pkg
    import paper_2411_04975_b200 as sfx
    w = get_workload(name)
    c = w.cfg
    B = c.batch
    sample = sorted({0, 1, 37 % B, B // 2 - 1, B // 2, (5 * B) // 7, B - 2, B - 1})
    dev = U.DEV
    store = sfx.SuffixStore(torch.as_tensor(w.corpus(), device=dev), torch.as_tensor(w.corpus_offsets(), device=dev),
                            vocab=c.vocab, depth_cap=c.depth_cap, max_requests=B, max_req_tokens=c.prompt_len + 64,
                            max_spec_cap=c.max_spec)
    prompts = [w.prompt(i) for i in range(B)]
    off, flat = U.ragged(prompts)
    slots = torch.arange(B, dtype=torch.int32, device=dev)
    if one_launch:
        store.build_requests(np.arange(B, dtype=np.int32), off, U.dev_i32(flat))
    else:
        store.append(slots, torch.as_tensor(off, device=dev), U.dev_i32(flat), torch.ones(B, dtype=torch.uint8, device=dev))
    ref = oracle_pkg.SuffixOracle(c.depth_cap, len(sample))
    ref.global_build(w.corpus(), w.corpus_offsets())
    ref.slot_append_batch(list(range(len(sample))), [prompts[i] for i in sample], n_threads=8)
    assert store.stats()["global_nodes"] == ref.node_count(-1)
    sched = accept_schedule(B, 3)
    cont = [w.continuation(i, prompts[i], length=int(sched[:, i].sum()) + 1) for i in range(B)]
    cur = np.zeros(B, dtype=np.int64)
    pending = None                                             # (offsets, tokens) accepted in the last step
    drafted = 0
    for step in range(3):
        if one_launch and pending is not None:
            out = store.step(slots, torch.as_tensor(pending[0], device=dev), U.dev_i32(pending[1]), c.max_pattern,
                             c.alpha, c.max_spec)
        else:
            out = store.speculate(slots, c.max_pattern, c.alpha, c.max_spec)
        torch.cuda.synchronize()
        got = {k: v.cpu().numpy() for k, v in out.items()}
        got["mask"] = got["mask"].view(np.uint32)
        want = ref.speculate(list(range(len(sample))), c.max_pattern, c.alpha, c.max_spec, n_threads=8)
        U.assert_same_drafts({k: v[sample] for k, v in got.items()}, want)
        _check_draft_properties(got, c, c.prompt_len + cur)
        drafted += int(got["n_draft"].sum())
        # next decode step
        a = sched[step]
        lists = [cont[i][cur[i]:cur[i] + a[i]] for i in range(B)]
        cur += a
        o2, f2 = U.ragged(lists)
        if one_launch and step < 2:
            pending = (o2, f2)                                  # appended by the next step's launch
        else:
            store.append(slots, torch.as_tensor(o2, device=dev), U.dev_i32(f2))
        ref.slot_append_batch(list(range(len(sample))), [lists[i] for i in sample], n_threads=8)
    assert drafted > 0
    # the sampled per-request trees, node by node (enumerated on the device)
    for k, i in enumerate(sample[:3]):
        _same_tree(U, store, i, ref, k)
    store.free()
    ref.close()


def _check_draft_properties(got, c, t_of):
    """What holds for every row of any batch: parents precede children, the mask of a node is its
    parent's plus its own bit, positions follow from the depth, padding is -1 / 0, the budget
    and the depth cap are respected."""
    n = got["n_draft"]
    B = len(n)
    assert (got["status"] == 0).all() and (n >= 0).all() and (n <= c.max_spec).all()
    assert ((got["score"] > 0) == (n > 0)).all() and (got["score"] <= n).all()
    for i in range(B):
        k = int(n[i])
        par = got["parents"][i, :k]
        assert (par < np.arange(k)).all() and (par >= -1).all()
        depth = np.zeros(k, dtype=np.int64)
        for j in range(k):
            depth[j] = 1 if par[j] < 0 else depth[par[j]] + 1
            row = int(got["mask"][i, j, 0]) | (int(got["mask"][i, j, 1]) << 32)
            prow = 0 if par[j] < 0 else int(got["mask"][i, par[j], 0]) | (int(got["mask"][i, par[j], 1]) << 32)
            assert row == prow | (1 << j)
        assert (got["positions"][i, :k] == int(t_of[i]) + depth - 1).all()
        assert (got["tokens"][i, k:] == -1).all() and (got["mask"][i, k:] == 0).all()
        assert k <= max(1, int(c.alpha * got["chosen_p"][i])) and depth.max(initial=0) <= c.depth_cap - got["chosen_p"][i]


def _same_tree(U, store, tree, ref, ref_tree):
    """Tree `tree` of the store, enumerated on the device, against tree `ref_tree` of the oracle."""
    depth, parent, tok, cnt = ref.dump(ref_tree)
    nn = len(tok)
    rec = {k: v.cpu().numpy() for k, v in store.enumerate(tree, nn + 8).items()}
    assert len(rec["token"]) == nn
    assert np.array_equal(U.canonical_nodes(rec["parent"], rec["token"], rec["count"], rec["depth"]),
                          U.canonical_nodes(parent, tok, cnt, depth))
    if tree >= 0:
        assert int(store.slot_info(U.dev_i32([tree]))["nodes"][0]) == nn


def test_closed_loop_full_size_sampled_against_oracle(U):
    """The closed-loop workload at full size (256 slots, 4,096-token prompts, 4 M-token global tree), 30 steps:
    speculate, simulated verification, append; finished outputs go into the global tree and
    their slots are refilled through sd_build_requests.  Outputs are kept short so that requests
    do finish within the 30 steps.  The oracle follows the global tree and a sample of the slots."""
    from workload.generator import get_workload
    from workload.closed_loop import ClosedLoop
    import oracle as oracle_pkg
    import paper_2411_04975_b200 as sfx
    w = get_workload("closed_loop")
    c = w.cfg
    B = c.batch
    dev = U.DEV
    sample = [0, 1, 50, 128, 200, 255]
    pos = {s: k for k, s in enumerate(sample)}
    store = sfx.SuffixStore(torch.as_tensor(w.corpus(), device=dev), torch.as_tensor(w.corpus_offsets(), device=dev),
                            vocab=c.vocab, depth_cap=c.depth_cap, max_requests=B, max_req_tokens=c.prompt_len + 128,
                            max_spec_cap=c.max_spec)
    ref = oracle_pkg.SuffixOracle(c.depth_cap, len(sample))
    ref.global_build(w.corpus(), w.corpus_offsets())
    loop = ClosedLoop(w, B, out_lo=12, out_hi=100)

    def apply(items):
        sl, lists, reset = items
        new = [i for i in range(len(sl)) if sl[i] >= 0 and reset[i]]
        keep = [i for i in range(len(sl)) if not (sl[i] >= 0 and reset[i])]
        if keep:
            o, f = U.ragged([lists[i] for i in keep])
            store.append(U.dev_i32([sl[i] for i in keep]), torch.as_tensor(o, device=dev),
                         U.dev_i32(f) if f.size else torch.zeros(0, dtype=torch.int32, device=dev))
        if new:
            o, f = U.ragged([lists[i] for i in new])
            store.build_requests(np.asarray([sl[i] for i in new], dtype=np.int32), o, U.dev_i32(f))
        for i in range(len(sl)):
            if sl[i] < 0:
                ref.global_insert(lists[i])
            elif sl[i] in pos:
                if reset[i]:
                    ref.slot_reset(pos[sl[i]])
                ref.slot_append_batch([pos[sl[i]]], [lists[i]])

    apply(loop.start())
    slots = torch.arange(B, dtype=torch.int32, device=dev)
    for step in range(30):
        out = store.speculate(slots, c.max_pattern, c.alpha, c.max_spec)
        torch.cuda.synchronize()
        got = {k: v.cpu().numpy() for k, v in out.items()}
        got["mask"] = got["mask"].view(np.uint32)
        want = ref.speculate(list(range(len(sample))), c.max_pattern, c.alpha, c.max_spec, n_threads=6)
        try:
            U.assert_same_drafts({k: v[sample] for k, v in got.items()}, want)
        except AssertionError as e:
            raise AssertionError(f"step {step}: {e}") from e
        t_of = store.slot_info(slots)["len"].cpu().numpy()
        _check_draft_properties(got, c, t_of)
        apply(loop.advance(got))
    s = loop.summary()
    assert s["finished_requests"] >= 20, s
    st = store.stats()
    assert st["global_nodes"] == ref.node_count(-1) and st["global_status"] == 0
    for k in (0, 3):
        _same_tree(U, store, sample[k], ref, k)
    store.free()
    ref.close()


# ---------------------------------------------------------------- sort-based per-request build (a2)
@pytest.mark.parametrize("D,vocab", [(1, 3), (4, 2), (7, 30), (32, 5), (32, 2000)])
def test_build_requests_equals_token_by_token_append(U, D, vocab):
    import paper_2411_04975_b200 as sfx
    rng = np.random.default_rng(D * 31 + vocab)
    n_slots = 9
    pr = U.Pair(_rand_seqs(rng, 4, 20, 100, vocab), vocab=vocab, D=D, n_slots=n_slots, max_req_tokens=3000)
    # slot 8 holds an older request that is replaced; slot 5 stays untouched
    pr.append([8, 5], _rand_seqs(rng, 2, 40, 80, vocab), reset=[1, 1])
    slots = [3, 8, 0, 7, 2]
    prompts = _rand_seqs(rng, 5, 0, 2500, vocab)
    prompts[2] = np.zeros(0, dtype=np.int32)                     # an empty prompt
    prompts[3] = np.full(300, vocab - 1, dtype=np.int32)         # one token repeated
    off, flat = U.ragged(prompts)
    pr.g.build_requests(slots, off, U.dev_i32(flat) if flat.size else torch.zeros(0, dtype=torch.int32, device=U.DEV))
    for s_, p_ in zip(slots, prompts):
        pr.o.slot_reset(s_)
        pr.o.slot_append(s_, p_)
    for s_ in range(n_slots):
        pr.check_tree(s_)
    pr.check_speculate(list(range(n_slots)), 32, 2.0, 64)
    # the trees keep growing token by token afterwards (offline runs are exact fits and must move)
    for step in range(3):
        pr.append(list(range(n_slots)), _rand_seqs(rng, n_slots, 0, 12, vocab))
        pr.check_speculate(list(range(n_slots)), 16, 1.5, 40)
    for s_ in range(n_slots):
        pr.check_tree(s_)
    # argument errors change nothing
    for bad in ([0, 0], [0, 99]):
        with pytest.raises(sfx.SuffixSpecError):
            pr.g.build_requests(bad, [0, 1, 2], U.dev_i32([0, 0]))
    with pytest.raises(sfx.SuffixSpecError):
        pr.g.build_requests([0], [0, 1], U.dev_i32([vocab]))
    pr.check_tree(0)
    pr.close()


def test_build_requests_long_and_short_prompts(U):
    """Prompts up to 16,384 tokens are sorted by one block each, longer ones by the general
    pipeline: both must give the tree of the token-by-token append."""
    rng = np.random.default_rng(5)
    vocab, D = 300, 12

    def text(L):
        s = np.minimum(rng.zipf(1.3, size=L) - 1, vocab - 1).astype(np.int32)
        if L > 64:
            s[L // 2:L // 2 + L // 8] = s[:L // 8]                # a long copy
            s[-40:] = 7                                           # a constant tail
        return s

    for lens in ([16384, 5, 0, 9000], [17000, 3], [1, 2, 4097]):
        pr = U.Pair([text(50)], vocab=vocab, D=D, n_slots=len(lens), max_req_tokens=max(lens) + 8)
        prompts = [text(L) for L in lens]
        off, flat = U.ragged(prompts)
        pr.g.build_requests(np.arange(len(lens), dtype=np.int32), off, U.dev_i32(flat))
        for q, p_ in enumerate(prompts):
            pr.o.slot_reset(q)
        pr.o.slot_append_batch(list(range(len(lens))), prompts, n_threads=4)
        for q in range(len(lens)):
            pr.check_tree(q)
        pr.check_speculate(list(range(len(lens))), 8, 2.0, 16)
        pr.close()


def test_build_requests_pool_overflow(U):
    rng = np.random.default_rng(8)
    pr = U.Pair([], vocab=500, D=8, n_slots=2, max_req_tokens=64, slot_pool_nodes=120)
    prompts = [rng.integers(0, 500, size=60).astype(np.int32), rng.integers(0, 500, size=10).astype(np.int32)]
    off, flat = U.ragged(prompts)
    pr.g.build_requests([0, 1], off, U.dev_i32(flat))
    info = pr.g.slot_info(U.dev_i32([0, 1]))
    assert int(info["status"][0]) == 2 and int(info["len"][0]) == 0 and int(info["nodes"][0]) == 0
    pr.o.slot_append(1, prompts[1])
    pr.check_tree(1)
    pr.close()


def test_entropy_matches_oracle(U):
    rng = np.random.default_rng(23)
    pr = U.Pair(_rand_seqs(rng, 30, 20, 400, 9) + [np.arange(2000, dtype=np.int32) % 700], vocab=700, D=12, n_slots=3,
                max_req_tokens=600)
    pr.append([0, 2, -1], _rand_seqs(rng, 3, 100, 500, 9), reset=[1, 1, 0])
    pr.append([0, -1], _rand_seqs(rng, 2, 50, 90, 700))
    for tree in (-1, 0, 1, 2):
        want = pr.o.entropy(tree)
        got = pr.g.entropy(tree)
        assert abs(got - want) <= 1e-9 * max(1.0, abs(want)), (tree, got, want)
    assert pr.g.entropy(1) == 0.0                                # empty slot
    pr.close()


# ---------------------------------------------------------------- fused decode step
@pytest.mark.parametrize("vocab,D", [(2, 32), (6, 8), (40, 16)])
def test_step_equals_append_then_speculate(U, vocab, D):
    rng = np.random.default_rng(vocab * 7 + D)
    n_slots = 20
    pr = U.Pair(_rand_seqs(rng, 15, 50, 300, vocab), vocab=vocab, D=D, n_slots=n_slots, max_req_tokens=400)
    pr.append(list(range(n_slots)), _rand_seqs(rng, n_slots, 0, 150, vocab), reset=[1] * n_slots)
    slots = list(range(n_slots))
    for step in range(6):
        lists = _rand_seqs(rng, n_slots, 0, 17, vocab)
        if step == 2:
            lists[3] = np.full(30, vocab - 1, dtype=np.int32)       # a repeated token
        off, flat = U.ragged(lists)
        out = pr.g.step(U.dev_i32(slots), torch.as_tensor(off, device=U.DEV),
                        U.dev_i32(flat) if flat.size else torch.zeros(0, dtype=torch.int32, device=U.DEV), 32, 2.0, 64,
                        flags=4 if step == 4 else 0)
        torch.cuda.synchronize()
        pr.o.slot_append_batch(slots, lists, n_threads=4)
        want = pr.o.speculate(slots, 32, 2.0, 64, M=64, flags=4 if step == 4 else 0, n_threads=4)
        got = {k: v.cpu().numpy() for k, v in out.items()}
        got["mask"] = got["mask"].view(np.uint32)
        U.assert_same_drafts(got, want)
        # plain speculate on the stepped store agrees too (the cached match nodes are consistent)
        pr.check_speculate(slots, 32, 2.0, 64)
    for s_ in range(n_slots):
        pr.check_tree(s_)
    pr.close()


def test_more_requests_than_block_slots(U):
    """Over 296 requests (two 16-warp blocks per SM on 148 SMs) the kernel runs with smaller blocks."""
    rng = np.random.default_rng(320)
    vocab, n_slots = 60, 330
    pr = U.Pair(_rand_seqs(rng, 12, 100, 400, vocab), vocab=vocab, D=32, n_slots=n_slots, max_req_tokens=200)
    slots = list(range(n_slots))
    pr.append(slots, _rand_seqs(rng, n_slots, 20, 90, vocab), reset=[1] * n_slots)
    pr.check_speculate(slots, 32, 2.0, 64)
    lists = _rand_seqs(rng, n_slots, 0, 9, vocab)
    off, flat = U.ragged(lists)
    out = pr.g.step(U.dev_i32(slots), torch.as_tensor(off, device=U.DEV), U.dev_i32(flat), 32, 2.0, 64)
    torch.cuda.synchronize()
    pr.o.slot_append_batch(slots, lists, n_threads=4)
    want = pr.o.speculate(slots, 32, 2.0, 64, M=64, n_threads=4)
    got = {k: v.cpu().numpy() for k, v in out.items()}
    got["mask"] = got["mask"].view(np.uint32)
    U.assert_same_drafts(got, want)
    pr.close()


def test_step_with_pinned_host_buffers(U):
    """Inputs and outputs in page-locked host memory: the kernel reads and writes them itself."""
    rng = np.random.default_rng(77)
    vocab, n_slots = 200, 12
    pr = U.Pair(_rand_seqs(rng, 10, 50, 200, vocab), vocab=vocab, D=16, n_slots=n_slots, max_req_tokens=300)
    pr.append(list(range(n_slots)), _rand_seqs(rng, n_slots, 20, 100, vocab), reset=[1] * n_slots)
    slots = list(range(n_slots))
    h_packed = torch.empty(pr.g.alloc_outputs(n_slots)["packed"].numel(), dtype=torch.uint8).pin_memory()
    h_out = pr.g.unpack_outputs(h_packed, n_slots)
    for step in range(3):
        lists = _rand_seqs(rng, n_slots, 0, 9, vocab)
        off, flat = U.ragged(lists)
        h_slots = torch.as_tensor(np.asarray(slots, dtype=np.int32)).pin_memory()
        h_off = torch.as_tensor(off).pin_memory()
        h_tok = torch.as_tensor(flat if flat.size else np.zeros(1, dtype=np.int32)).pin_memory()
        h_packed.fill_(0x5A)
        if step == 1:                                               # the pre-marshalled form of the same call
            pr.g.bind_step(h_slots, h_off, h_tok, 16, 2.0, 32, 0, None, h_out)()
        else:
            pr.g.step(h_slots, h_off, h_tok[:flat.size], 16, 2.0, 32, 0, None, h_out)
        torch.cuda.synchronize()
        pr.o.slot_append_batch(slots, lists, n_threads=2)
        want = pr.o.speculate(slots, 16, 2.0, 32, M=64, n_threads=2)
        got = {k: v.numpy().copy() for k, v in h_out.items()}
        got["mask"] = got["mask"].view(np.uint32)
        U.assert_same_drafts(got, want)
    pr.close()


def test_step_reports_a_stopped_append(U):
    rng = np.random.default_rng(4)
    pr = U.Pair(_rand_seqs(rng, 3, 30, 60, 50), vocab=50, D=8, n_slots=3, max_req_tokens=40)
    pr.append([0, 1, 2], _rand_seqs(rng, 3, 10, 20, 50), reset=[1, 1, 1])
    lists = [rng.integers(0, 50, size=60).astype(np.int32),        # overflows the text buffer of slot 0
             np.array([3, 99], dtype=np.int32),                      # token outside the vocabulary
             rng.integers(0, 50, size=4).astype(np.int32)]
    off, flat = U.ragged(lists)
    out = pr.g.step(U.dev_i32([0, 1, 2]), torch.as_tensor(off, device=U.DEV), U.dev_i32(flat), 8, 2.0, 16)
    torch.cuda.synchronize()
    st = out["status"].cpu().numpy()
    assert st[0] & 2 and st[1] & 8 and st[2] == 0
    assert int(out["n_draft"][0]) == 0 and int(out["n_draft"][1]) == 0
    pr.o.slot_append(2, lists[2])
    want = pr.o.speculate([2], 8, 2.0, 16, M=64)
    assert int(out["n_draft"][2]) == int(want["n_draft"][0])
    assert out["tokens"][2].cpu().numpy().tolist() == want["tokens"][0].tolist()
    pr.close()


# ---------------------------------------------------------------- score threshold, duplicate slots, allocation failures
def test_score_threshold_is_strict_on_the_gpu(U):
    """Section 3.2: the chosen tree is used only if SCORE > tau.  Thresholds just below, at and just
    above a score that really occurs: sd_speculate, sd_step and sd_speculate_noalloc against the oracle."""
    import paper_2411_04975_b200 as sfx
    rng = np.random.default_rng(41)
    n = 24
    pr = U.Pair(_rand_seqs(rng, 12, 80, 300, 6), vocab=6, D=16, n_slots=n, max_req_tokens=200)
    pr.append(list(range(n)), _rand_seqs(rng, n, 20, 120, 6), reset=[1] * n)
    slots = list(range(n))
    got0, _ = pr.check_speculate(slots, 16, 2.0, 48)
    pos = np.sort(got0["score"][got0["score"] > 0])
    assert pos.size >= 8
    s = float(pos[pos.size // 2])
    empty = torch.zeros(0, dtype=torch.int32, device=U.DEV)
    no_new = torch.zeros(n + 1, dtype=torch.int64, device=U.DEV)
    for tau in (float(np.nextafter(s, 0.0)), s, float(np.nextafter(s, np.inf)), 1e9):
        got, want = pr.check_speculate(slots, 16, 2.0, 48, tau=tau)
        keep = got0["score"] > tau                               # strictly above: kept unchanged
        assert np.array_equal(got["n_draft"][keep], got0["n_draft"][keep])
        assert (got["n_draft"][~keep] == 0).all() and (got["chosen_tree"][~keep] == -1).all()
        assert (got["score"][~keep] == 0).all() and (got["tokens"][~keep] == -1).all()
        out = pr.g.step(U.dev_i32(slots), no_new, empty, 16, 2.0, 48, tau=tau)
        alt = pr.g.alloc_outputs(n)
        sfx.sd_speculate_noalloc(pr.g.handle, U.dev_i32(slots), 16, 2.0, 48, 0, None, alt, tau)
        torch.cuda.synchronize()
        for o in (out, alt):
            g = {k: v.cpu().numpy() for k, v in o.items()}
            g["mask"] = g["mask"].view(np.uint32)
            U.assert_same_drafts(g, want)
    assert (got0["score"] > float(np.nextafter(s, 0.0))).sum() == (got0["score"] > s).sum() + (got0["score"] == s).sum()
    for bad in (-1.0, float("nan")):
        with pytest.raises(sfx.SuffixSpecError):
            pr.g.speculate(U.dev_i32(slots), 16, 2.0, 48, tau=bad)
    pr.close()


def test_a_slot_that_appears_twice_is_refused(U):
    """Two blocks on one tree would race: every later appearance of a slot gets the bad-slot status
    and no draft, in sd_speculate and in sd_step (whose extra tokens are not appended either)."""
    rng = np.random.default_rng(43)
    pr = U.Pair(_rand_seqs(rng, 8, 50, 200, 5), vocab=5, D=12, n_slots=8, max_req_tokens=300)
    pr.append(list(range(6)), _rand_seqs(rng, 6, 30, 100, 5), reset=[1] * 6)
    call = [0, 1, 0, 2, 1, 0, 5]
    first = [0, 1, 3, 6]                                         # rows that are first appearances
    out = pr.g.speculate(U.dev_i32(call), 12, 2.0, 40)
    torch.cuda.synchronize()
    got = {k: v.cpu().numpy() for k, v in out.items()}
    got["mask"] = got["mask"].view(np.uint32)
    assert got["status"].tolist() == [0, 0, 1, 0, 1, 1, 0]
    assert (got["n_draft"][[2, 4, 5]] == 0).all() and (got["chosen_tree"][[2, 4, 5]] == -1).all()
    want = pr.o.speculate([call[i] for i in first], 12, 2.0, 40, M=64)
    U.assert_same_drafts({k: v[first] for k, v in got.items()}, want)
    # one-launch step: only the first appearance appends
    lists = _rand_seqs(rng, len(call), 1, 6, 5)
    off, flat = U.ragged(lists)
    out = pr.g.step(U.dev_i32(call), torch.as_tensor(off, device=U.DEV), U.dev_i32(flat), 12, 2.0, 40)
    torch.cuda.synchronize()
    got = {k: v.cpu().numpy() for k, v in out.items()}
    got["mask"] = got["mask"].view(np.uint32)
    assert got["status"].tolist() == [0, 0, 1, 0, 1, 1, 0]
    pr.o.slot_append_batch([call[i] for i in first], [lists[i] for i in first])
    want = pr.o.speculate([call[i] for i in first], 12, 2.0, 40, M=64)
    U.assert_same_drafts({k: v[first] for k, v in got.items()}, want)
    for s in range(6):
        pr.check_tree(s)
    pr.close()


@pytest.mark.parametrize("n_slots", [3, 200, 310])
def test_text_too_long_for_shared_memory_goes_through_the_tree(U, n_slots):
    """A store whose text buffer (max_req_tokens) is larger than the shared memory a block can give
    it: nothing is staged, every per-request job goes through the request's tree and, in sd_step,
    waits for the append.  One, two and four blocks per SM."""
    rng = np.random.default_rng(53 + n_slots)
    pr = U.Pair(_rand_seqs(rng, 10, 60, 300, 7), vocab=7, D=16, n_slots=n_slots, max_req_tokens=40000,
                slot_pool_nodes=6000)
    slots = list(range(n_slots))
    pr.append(slots, _rand_seqs(rng, n_slots, 0, 150, 7), reset=[1] * n_slots)
    pr.check_speculate(slots, 16, 2.0, 48)
    for _ in range(3):
        lists = _rand_seqs(rng, n_slots, 0, 9, 7)
        off, flat = U.ragged(lists)
        out = pr.g.step(U.dev_i32(slots), torch.as_tensor(off, device=U.DEV),
                        U.dev_i32(flat) if flat.size else torch.zeros(0, dtype=torch.int32, device=U.DEV), 16, 2.0, 48)
        torch.cuda.synchronize()
        pr.o.slot_append_batch(slots, lists, n_threads=4)
        want = pr.o.speculate(slots, 16, 2.0, 48, M=64, n_threads=4)
        got = {k: v.cpu().numpy() for k, v in out.items()}
        got["mask"] = got["mask"].view(np.uint32)
        U.assert_same_drafts(got, want)
    pr.check_tree(0)
    pr.check_tree(n_slots - 1)
    pr.close()


def test_device_allocation_failures_are_error_codes(U):
    """Every device allocation of sd_build and sd_build_requests fails once (test hook of the
    library): the call returns the out-of-memory code, nothing leaks, and the next call works."""
    import paper_2411_04975_b200 as sfx
    rng = np.random.default_rng(47)
    corpus = _rand_seqs(rng, 6, 40, 120, 7)
    off, flat = U.ragged(corpus)
    lib = sfx.library()
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]

    def build():
        return sfx.SuffixStore(U.dev_i32(flat), torch.as_tensor(off, device=U.DEV), vocab=7, depth_cap=8,
                               max_requests=4, max_req_tokens=128, max_spec_cap=32)
    failed = 0
    try:
        for k in range(1, 80):
            lib.sd_debug_fail_alloc(k)
            try:
                store = build()
            except sfx.SuffixSpecError as e:
                assert e.code == -3, e
                failed += 1
                continue
            store.free()                                         # the k-th allocation was optional, or there is none
        assert failed >= 5
        lib.sd_debug_fail_alloc(0)
        torch.cuda.synchronize()
        assert abs(torch.cuda.mem_get_info()[0] - free0) <= (8 << 20)       # nothing left behind
        # prompts through sd_build_requests with failing workspace allocations, then for real
        pr = U.Pair(corpus, vocab=7, D=8, n_slots=4, max_req_tokens=128, M=32)
        prompts = _rand_seqs(rng, 4, 10, 90, 7)
        poff, pflat = U.ragged(prompts)
        refused = 0
        for k in range(1, 40):
            lib.sd_debug_fail_alloc(k)
            try:
                pr.g.build_requests(np.arange(4, dtype=np.int32), poff, U.dev_i32(pflat))
            except sfx.SuffixSpecError as e:
                assert e.code == -3, e
                refused += 1
        lib.sd_debug_fail_alloc(0)
        assert refused >= 1
        pr.g.build_requests(np.arange(4, dtype=np.int32), poff, U.dev_i32(pflat))
        for s in range(4):
            pr.o.slot_reset(s)
        pr.o.slot_append_batch(list(range(4)), prompts)
        for s in range(4):
            pr.check_tree(s)
        pr.check_speculate([0, 1, 2, 3], 8, 2.0, 32)
        pr.close()
    finally:
        lib.sd_debug_fail_alloc(0)
