"""Host-side checks that need no GPU: the seeded generator, the closed-loop
harness, and that the CUDA library loads and exports the declared C ABI."""
import ctypes
import os
import re

import numpy as np

from workload.closed_loop import accept_longest_path
from workload.generator import CONFIGS, accept_schedule, get_workload, splitmix_block

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_splitmix64_reference_values():
    # SplitMix64 with seed 0: first outputs of the published generator
    got = splitmix_block(0, 3)
    assert [int(x) for x in got] == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_generator_is_deterministic_and_has_the_configured_shape():
    w1, w2 = get_workload("tiny"), get_workload("tiny")
    c = w1.cfg
    a, b = w1.corpus(), w2.corpus()
    assert a.dtype == np.int32 and a.shape == (c.n_seqs * c.seq_len,) and np.array_equal(a, b)
    assert a.min() >= 0 and a.max() < c.vocab
    p = w1.prompt(3)
    assert p.shape == (c.prompt_len,) and np.array_equal(p, w2.prompt(3)) and not np.array_equal(p, w1.prompt(4))
    cont = w1.continuation(3, p)
    assert c.out_len_lo <= len(cont) <= c.out_len_hi
    # repetition: most 8-grams of the corpus occur more than once (copy probability 0.7)
    grams = np.lib.stride_tricks.sliding_window_view(a[:8192], 8)
    _, counts = np.unique(grams, axis=0, return_counts=True)
    assert (counts > 1).sum() > 0
    assert set(CONFIGS) == {"tiny", "agentic", "large_batch", "low_repetition", "closed_loop"}
    assert CONFIGS["large_batch"].batch == 256 and CONFIGS["large_batch"].n_seqs * CONFIGS["large_batch"].seq_len == 4194304


def test_accept_schedule():
    s = accept_schedule(256, 50)
    assert s.shape == (50, 256) and s.min() >= 1 and s.max() <= 16 and 3.0 < s.mean() < 5.0
    assert np.array_equal(s, accept_schedule(256, 50))


def test_simulated_verifier_accepts_the_matching_path():
    #        root -> 5 -> 6 -> 7
    #             -> 9 -> 6
    tokens = np.array([5, 9, 6, 6, 7]); parents = np.array([-1, -1, 0, 1, 2])
    assert accept_longest_path(tokens, parents, 5, np.array([5, 6, 7, 1])) == 3
    assert accept_longest_path(tokens, parents, 5, np.array([9, 6, 7])) == 2
    assert accept_longest_path(tokens, parents, 5, np.array([4])) == 0
    assert accept_longest_path(tokens, parents, 0, np.array([5])) == 0
    assert accept_longest_path(tokens, parents, 5, np.array([5, 6])) == 2      # truth ends first


def test_library_loads_and_exports_every_declared_symbol():
    from paper_2411_04975_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    header = open(os.path.join(ROOT, "include", "suffixspec.h")).read()
    declared = set(re.findall(r"^\w[\w\s\*]*?\b(sd_\w+)\s*\(", header, flags=re.M))
    assert {"sd_build", "sd_append", "sd_speculate", "sd_free"} <= declared
    for name in declared:
        assert hasattr(lib, name), name
    lib.sd_strerror.restype = ctypes.c_char_p
    assert lib.sd_strerror(0) == b"ok" and lib.sd_strerror(-4) == b"capacity exceeded"
    # host-side argument checks need no device
    assert lib.sd_build(None, None, None, 0, None, None) == -1
    lib.sd_free(None)


def test_bench_reference_arm_prints_the_contract_line():
    """`bench.py --impl reference` (the CPU oracle timed on the host) needs no GPU: one JSON line
    with the keys of the bench contract."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    p = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--config", "tiny",
                        "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=300, cwd=root)
    assert p.returncode == 0, p.stderr[-2000:]
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "trees/s" and line["higher_is_better"] is True
    assert line["value"] > 0 and line["steps"] == 2 and line["warmup"] == 1 and line["n_gpus"] == 1
    assert line["config"]["workload"] == "tiny" and "batch 8" in line["metric"]
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": "trees/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
