"""Seeded synthetic workloads for batched suffix-tree draft generation.

This module only makes token arrays.  It holds none of the method's arithmetic
(no tries, no scores) so that the CPU oracle and the CUDA path can both be fed
from it without sharing any logic.

Text model.  Agentic LLM traffic is dominated by long spans that repeat
earlier text (Section 2, "Agentic AI Algorithms"; Section 4.2, the discussion
of the speculation-tree example).  A sequence is therefore produced event by
event: with probability ``copy_prob`` an event copies a span whose start is
uniform over all text generated so far in the pool and whose length is
geometric with mean ``mean_span``; otherwise it emits one fresh token drawn
from a Zipf(s) law over a seeded permutation of the vocabulary.

Random numbers.  One counter-based generator (SplitMix64, Steele, Lea and
Flood 2014): the k-th output of a stream with seed ``s`` is
``mix(s + (k + 1) * GOLDEN)``.  Streams are keyed by (master seed, config id,
purpose, index), so any sequence can be regenerated on its own.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional

import numpy as np

MASTER_SEED = 20241104
_GOLDEN = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_MASK = (1 << 64) - 1

PURPOSE_PERM = 1
PURPOSE_CORPUS = 2
PURPOSE_PROMPT = 3
PURPOSE_CONT = 4
PURPOSE_OUTLEN = 5


def _mix(z: int) -> int:
    z &= _MASK
    z = ((z ^ (z >> 30)) * _M1) & _MASK
    z = ((z ^ (z >> 27)) * _M2) & _MASK
    return z ^ (z >> 31)


def stream_seed(config_id: int, purpose: int, index: int, master: int = MASTER_SEED) -> int:
    s = _mix(master + _GOLDEN)
    s = _mix(s ^ ((config_id + 1) * 0xD1B54A32D192ED03 & _MASK))
    s = _mix(s ^ ((purpose + 1) * 0x8CB92BA72F3D8DD7 & _MASK))
    s = _mix(s ^ ((index + 1) * 0xABC98388FB8FAC03 & _MASK))
    return s


def splitmix_block(seed: int, n: int) -> np.ndarray:
    """First ``n`` outputs of the stream ``seed`` as uint64."""
    with np.errstate(over="ignore"):
        k = np.arange(1, n + 1, dtype=np.uint64)
        z = np.uint64(seed) + k * np.uint64(_GOLDEN)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(_M1)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(_M2)
        z = z ^ (z >> np.uint64(31))
    return z


def _unit(u64: np.ndarray) -> np.ndarray:
    """uint64 -> float64 in [0, 1) from the top 53 bits."""
    return (u64 >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


class Vocabulary:
    """Zipf(s) over ranks 1..V, ranks mapped to token ids by a seeded shuffle."""

    def __init__(self, vocab: int, zipf_s: float, config_id: int):
        self.vocab = vocab
        w = np.arange(1, vocab + 1, dtype=np.float64) ** (-zipf_s)
        cdf = np.cumsum(w)
        self.cdf = cdf / cdf[-1]
        # Fisher-Yates with the counter-based stream.
        r = splitmix_block(stream_seed(config_id, PURPOSE_PERM, 0), vocab)
        perm = np.arange(vocab, dtype=np.int32)
        for i in range(vocab - 1, 0, -1):
            j = int(r[i] % np.uint64(i + 1))
            perm[i], perm[j] = perm[j], perm[i]
        self.perm = perm

    def fresh(self, u: float) -> int:
        rank = int(np.searchsorted(self.cdf, u, side="right"))
        if rank >= self.vocab:
            rank = self.vocab - 1
        return int(self.perm[rank])


class _Pool:
    """Earlier text a copy event may draw from: a list of read-only segments
    (each a flat array cut into fixed-length sequences) plus the sequence being
    written."""

    def __init__(self):
        self.segs: List[tuple] = []   # (array, seq_len)
        self.total = 0

    def add(self, arr: np.ndarray, seq_len: int):
        if arr.size:
            self.segs.append((arr, seq_len, self.total))
            self.total += int(arr.size)

    def locate(self, g: int):
        """global index -> (array, start, end_of_its_sequence)"""
        for arr, seq_len, base in self.segs:
            if g < base + arr.size:
                o = g - base
                end = min((o // seq_len + 1) * seq_len, arr.size)
                return arr, o, end
        raise IndexError(g)


def _geometric(u: float, mean: float) -> int:
    if mean <= 1.0:
        return 1
    p = 1.0 / mean
    return 1 + int(math.floor(math.log(1.0 - u) / math.log(1.0 - p)))


def generate_sequence(length: int, vocab: Vocabulary, pool: _Pool, copy_prob: float,
                      mean_span: float, seed: int, corpus_prob: Optional[float] = None,
                      own_prefix: Optional[np.ndarray] = None) -> np.ndarray:
    """One sequence of ``length`` tokens.

    ``pool`` is the read-only earlier text; the sequence's own already-written
    part (preceded by ``own_prefix`` if given, e.g. the prompt of a
    continuation) is part of the copy pool too.  If ``corpus_prob`` is given,
    each event first decides with that probability to copy a span from the
    read-only pool only; otherwise the event is an ordinary one restricted to
    the sequence's own text and fresh tokens.
    """
    out = np.empty(length, dtype=np.int32)
    if own_prefix is None:
        own_prefix = np.empty(0, dtype=np.int32)
    npre = int(own_prefix.size)
    r = _unit(splitmix_block(seed, 4 * length + 8))
    k = 0
    n = 0
    while n < length:
        u_kind, u_src, u_len, u_tok = r[k], r[k + 1], r[k + 2], r[k + 3]
        k += 4
        own = npre + n
        if corpus_prob is not None:
            if u_kind < corpus_prob and pool.total > 0:
                avail, lo = pool.total, 0                  # corpus span
            else:
                # ordinary event on own text: reuse u_kind's remaining mass
                u2 = (u_kind - corpus_prob) / (1.0 - corpus_prob) if u_kind >= corpus_prob else 1.0
                if u2 < copy_prob and own > 0:
                    avail, lo = own, pool.total
                else:
                    avail = 0
                    lo = 0
        else:
            if u_kind < copy_prob and (pool.total + own) > 0:
                avail, lo = pool.total + own, 0
            else:
                avail, lo = 0, 0
        if avail == 0:
            out[n] = vocab.fresh(u_tok)
            n += 1
            continue
        g = lo + min(int(u_src * avail), avail - 1)
        span = _geometric(u_len, mean_span)
        if g < pool.total:
            arr, o, end = pool.locate(g)
            take = min(span, end - o, length - n)
            out[n:n + take] = arr[o:o + take]
        else:
            o = g - pool.total                            # index into prefix+own
            end = own
            take = min(span, end - o, length - n)
            if o + take <= npre:
                out[n:n + take] = own_prefix[o:o + take]
            else:
                for i in range(take):                     # may straddle prefix/own
                    q = o + i
                    out[n + i] = own_prefix[q] if q < npre else out[q - npre]
        n += take
    return out


@dataclasses.dataclass(frozen=True)
class WorkloadConfig:
    name: str
    config_id: int
    vocab: int
    n_seqs: int
    seq_len: int
    copy_prob: float
    mean_span: float
    depth_cap: int          # D
    batch: int              # B
    prompt_len: int
    max_pattern: int        # P
    alpha: float
    max_spec: int           # MAX_SPEC cap
    zipf_s: float = 1.1
    prompt_corpus_prob: Optional[float] = None
    out_len_lo: int = 128
    out_len_hi: int = 512
    steps: int = 0          # closed-loop steps (0: not a closed-loop config)

    def scaled(self, **kw) -> "WorkloadConfig":
        return dataclasses.replace(self, **kw)


CONFIGS = {
    "tiny": WorkloadConfig("tiny", 0, 32000, 64, 512, 0.7, 32.0, 32, 8, 256, 16, 1.0, 32),
    "agentic": WorkloadConfig("agentic", 1, 32000, 4000, 1024, 0.8, 48.0, 32, 64, 8192, 24, 2.0, 64,
                              prompt_corpus_prob=0.5),
    "large_batch": WorkloadConfig("large_batch", 2, 128256, 4096, 1024, 0.7, 32.0, 32, 256, 4096, 32,
                                  2.0, 64),
    "low_repetition": WorkloadConfig("low_repetition", 3, 128256, 4096, 1024, 0.15, 8.0, 32, 512, 4096,
                                     32, 2.0, 64),
    "closed_loop": WorkloadConfig("closed_loop", 4, 128256, 4096, 1024, 0.7, 32.0, 32, 256, 4096, 32,
                                  2.0, 64, steps=1000),
}


class Workload:
    """Corpus, prompts and (for the closed loop) hidden continuations."""

    def __init__(self, cfg: WorkloadConfig):
        self.cfg = cfg
        self.vocab = Vocabulary(cfg.vocab, cfg.zipf_s, cfg.config_id)
        self._corpus: Optional[np.ndarray] = None

    # ---- global corpus -------------------------------------------------
    def corpus(self) -> np.ndarray:
        """int32[n_seqs * seq_len]; sequence j is [j*seq_len, (j+1)*seq_len)."""
        if self._corpus is None:
            c = self.cfg
            flat = np.empty(c.n_seqs * c.seq_len, dtype=np.int32)
            for j in range(c.n_seqs):
                pool = _Pool()
                pool.add(flat[: j * c.seq_len], c.seq_len)
                flat[j * c.seq_len:(j + 1) * c.seq_len] = generate_sequence(
                    c.seq_len, self.vocab, pool, c.copy_prob, c.mean_span,
                    stream_seed(c.config_id, PURPOSE_CORPUS, j))
            self._corpus = flat
        return self._corpus

    def corpus_offsets(self) -> np.ndarray:
        c = self.cfg
        return np.arange(c.n_seqs + 1, dtype=np.int64) * c.seq_len

    def _corpus_pool(self) -> _Pool:
        pool = _Pool()
        pool.add(self.corpus(), self.cfg.seq_len)
        return pool

    # ---- prompts -------------------------------------------------------
    def prompt(self, index: int, length: Optional[int] = None) -> np.ndarray:
        c = self.cfg
        return generate_sequence(
            c.prompt_len if length is None else length, self.vocab, self._corpus_pool(),
            c.copy_prob, c.mean_span, stream_seed(c.config_id, PURPOSE_PROMPT, index),
            corpus_prob=c.prompt_corpus_prob)

    def prompts(self, n: Optional[int] = None) -> List[np.ndarray]:
        return [self.prompt(i) for i in range(self.cfg.batch if n is None else n)]

    # ---- closed loop ---------------------------------------------------
    def output_length(self, index: int) -> int:
        c = self.cfg
        u = _unit(splitmix_block(stream_seed(c.config_id, PURPOSE_OUTLEN, index), 1))[0]
        return c.out_len_lo + min(int(u * (c.out_len_hi - c.out_len_lo + 1)), c.out_len_hi - c.out_len_lo)

    def continuation(self, index: int, prompt: np.ndarray, length: Optional[int] = None) -> np.ndarray:
        """Hidden ground-truth output of request ``index`` (pool: corpus + its
        prompt + the continuation written so far)."""
        c = self.cfg
        return generate_sequence(
            self.output_length(index) if length is None else length, self.vocab,
            self._corpus_pool(), c.copy_prob, c.mean_span,
            stream_seed(c.config_id, PURPOSE_CONT, index), own_prefix=prompt)


def get_workload(name: str, **overrides) -> Workload:
    cfg = CONFIGS[name]
    if overrides:
        cfg = cfg.scaled(**overrides)
    return Workload(cfg)


def accept_schedule(n_requests: int, n_steps: int, seed_index: int = 0, mean_extra: float = 3.0,
                    cap: int = 16) -> np.ndarray:
    """int32[n_steps][n_requests]: tokens appended per request per decode step in
    the open-loop benchmark (1 bonus token + a geometric number of accepted
    drafts, capped), from the counter-based generator."""
    u = _unit(splitmix_block(stream_seed(99, PURPOSE_OUTLEN, seed_index), n_requests * n_steps))
    p = 1.0 / (mean_extra + 1.0)
    extra = np.floor(np.log1p(-u) / math.log(1.0 - p)).astype(np.int64)
    return (1 + np.minimum(extra, cap - 1)).astype(np.int32).reshape(n_steps, n_requests)
