"""sd_speculate_noalloc against sd_speculate.

The no-alloc entry point exists for hosts that cannot call the CUDA allocator
(a server that already owns all device memory, a plug-in handed only buffers
and a stream).  It keeps its scratch in a fixed array inside the library, shared
by all calls, so this test calls it twice in a row with different batches and
checks that nothing left in the array by the first call leaks into the second.
Collected last on purpose: if it fails, every other test has already run.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _same(a, b):
    for k in a:
        if k != "packed":                          # the buffer behind the views (has padding bytes)
            assert torch.equal(a[k], b[k]), k      # integers and fp64 score bits alike: exact


def test_noalloc_matches_sd_speculate_twice_in_a_row():
    import gpu_util as U
    import paper_2411_04975_b200 as sfx

    rng = np.random.default_rng(77)
    vocab, D, n_slots = 6, 32, 64
    corpus = [rng.integers(0, vocab, size=int(rng.integers(50, 400))).astype(np.int32) for _ in range(20)]
    pr = U.Pair(corpus, vocab=vocab, D=D, n_slots=n_slots, max_req_tokens=300)
    pr.append(list(range(n_slots)), [rng.integers(0, vocab, size=int(rng.integers(0, 200))).astype(np.int32)
                                     for _ in range(n_slots)], reset=[1] * n_slots)
    g = pr.g

    # call 1: the largest batch the fixed array takes (64 requests x 2 trees x depth 32 = 4096 jobs)
    slots = U.dev_i32(list(range(n_slots)))
    want = g.speculate(slots, 32, 2.0, 64)
    got = g.alloc_outputs(n_slots)
    sfx.sd_speculate_noalloc(g.handle, slots, 32, 2.0, 64, 0, None, got)
    torch.cuda.synchronize()
    _same(want, got)
    assert int(got["n_draft"].sum()) > 0

    # the trees move on, then call 2: a smaller batch in another order with other parameters;
    # the array still holds call 1's records
    pr.append(list(range(n_slots)), [rng.integers(0, vocab, size=3).astype(np.int32) for _ in range(n_slots)])
    slots2 = U.dev_i32([9, 3, 40, 11, 0])
    want2 = g.speculate(slots2, 7, 1.5, 20, sfx.FLAG_REQUEST_ONLY)
    got2 = g.alloc_outputs(5)
    sfx.sd_speculate_noalloc(g.handle, slots2, 7, 1.5, 20, sfx.FLAG_REQUEST_ONLY, None, got2)
    torch.cuda.synchronize()
    _same(want2, got2)
    # and the oracle agrees with both
    ref = pr.o.speculate([9, 3, 40, 11, 0], 7, 1.5, 20, M=64, flags=2)
    g2 = {k: v.cpu().numpy() for k, v in got2.items()}
    g2["mask"] = g2["mask"].view(np.uint32)
    U.assert_same_drafts(g2, ref)
    pr.close()


def test_noalloc_rejects_batches_beyond_its_fixed_array():
    import gpu_util as U
    import paper_2411_04975_b200 as sfx

    pr = U.Pair([np.arange(40, dtype=np.int32) % 5], vocab=5, D=32, n_slots=65, max_req_tokens=16)
    out = pr.g.alloc_outputs(65)
    with pytest.raises(sfx.SuffixSpecError) as e:
        sfx.sd_speculate_noalloc(pr.g.handle, U.dev_i32(list(range(65))), 8, 2.0, 64, 0, None, out)
    assert e.value.code == -4 and "capacity" in str(e.value)
    sfx.sd_speculate_noalloc(pr.g.handle, U.dev_i32(list(range(64))), 8, 2.0, 64, 0, None, pr.g.alloc_outputs(64))
    torch.cuda.synchronize()
    pr.close()
