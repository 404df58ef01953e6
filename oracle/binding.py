"""ctypes binding of the CPU oracle (test infrastructure only)."""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "suffix_oracle.cpp")
_LIB = os.path.join(_HERE, "libsuffix_oracle.so")

FLAG_GLOBAL_ONLY = 1
FLAG_REQUEST_ONLY = 2
FLAG_LINEAR = 4


def library_path() -> str:
    return _LIB


def build(force: bool = False) -> str:
    """Compile the oracle.  -ffp-contract=off keeps fp64 products and sums
    un-fused, as the scoring rules require."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread",
                               "-ffp-contract=off", "-o", _LIB, _SRC])
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        p32, p64, pd, pu32 = (C.POINTER(C.c_int32), C.POINTER(C.c_int64), C.POINTER(C.c_double),
                              C.POINTER(C.c_uint32))
        lib.sfx_oracle_create.restype = C.c_void_p
        lib.sfx_oracle_create.argtypes = [C.c_int, C.c_int]
        lib.sfx_oracle_destroy.argtypes = [C.c_void_p]
        lib.sfx_oracle_global_insert.argtypes = [C.c_void_p, p32, C.c_int64]
        lib.sfx_oracle_slot_reset.argtypes = [C.c_void_p, C.c_int]
        lib.sfx_oracle_slot_append.argtypes = [C.c_void_p, C.c_int, p32, C.c_int64]
        lib.sfx_oracle_slot_append_batch.argtypes = [C.c_void_p, C.c_int, p32, p64, p32, C.c_int]
        lib.sfx_oracle_slot_len.restype = C.c_int64
        lib.sfx_oracle_slot_len.argtypes = [C.c_void_p, C.c_int]
        lib.sfx_oracle_slot_updates.restype = C.c_int64
        lib.sfx_oracle_slot_updates.argtypes = [C.c_void_p, C.c_int]
        lib.sfx_oracle_slot_text.argtypes = [C.c_void_p, C.c_int, p32]
        lib.sfx_oracle_count.restype = C.c_int64
        lib.sfx_oracle_count.argtypes = [C.c_void_p, C.c_int, p32, C.c_int]
        lib.sfx_oracle_node_count.restype = C.c_int64
        lib.sfx_oracle_node_count.argtypes = [C.c_void_p, C.c_int]
        lib.sfx_oracle_dump.restype = C.c_int64
        lib.sfx_oracle_dump.argtypes = [C.c_void_p, C.c_int, C.c_int64, p32, p32, p32, p32]
        lib.sfx_oracle_candidate.restype = C.c_int
        lib.sfx_oracle_candidate.argtypes = [C.c_void_p, C.c_int, p32, C.c_int64, C.c_int, C.c_int, C.c_int,
                                             p32, p32, pd, pd]
        lib.sfx_oracle_entropy.restype = C.c_double
        lib.sfx_oracle_entropy.argtypes = [C.c_void_p, C.c_int]
        lib.sfx_oracle_budget.restype = C.c_int
        lib.sfx_oracle_budget.argtypes = [C.c_double, C.c_int, C.c_int]
        lib.sfx_oracle_speculate.argtypes = [C.c_void_p, C.c_int, p32, C.c_int, C.c_double, C.c_int, C.c_int,
                                             C.c_int, p32, p32, p32, p32, p32, pu32, p32, p32, pd, p64, C.c_int, C.c_double]
        _lib = lib
    return _lib


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a: np.ndarray, t):
    return a.ctypes.data_as(C.POINTER(t))


class SuffixOracle:
    """Global tree + per-request trees (slots) + Algorithm 1, on the CPU."""

    GLOBAL = -1

    def __init__(self, depth_cap: int, n_slots: int):
        self._lib = _load()
        self.D = depth_cap
        self.n_slots = n_slots
        self._h = C.c_void_p(self._lib.sfx_oracle_create(depth_cap, n_slots))

    def close(self):
        if self._h:
            self._lib.sfx_oracle_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- store ---------------------------------------------------------
    def global_insert(self, tokens) -> None:
        t = _i32(tokens)
        self._lib.sfx_oracle_global_insert(self._h, _p(t, C.c_int32), t.size)

    def global_build(self, corpus, offsets) -> None:
        corpus = _i32(corpus)
        for j in range(len(offsets) - 1):
            self.global_insert(corpus[int(offsets[j]):int(offsets[j + 1])])

    def slot_reset(self, slot: int) -> None:
        self._lib.sfx_oracle_slot_reset(self._h, slot)

    def slot_append(self, slot: int, tokens) -> None:
        t = _i32(tokens)
        self._lib.sfx_oracle_slot_append(self._h, slot, _p(t, C.c_int32), t.size)

    def slot_append_batch(self, slots, token_lists: Sequence, n_threads: int = 1) -> None:
        slots = _i32(slots)
        off = np.zeros(len(token_lists) + 1, dtype=np.int64)
        off[1:] = np.cumsum([len(t) for t in token_lists])
        flat = _i32(np.concatenate([_i32(t) for t in token_lists])) if len(token_lists) else _i32([])
        self._lib.sfx_oracle_slot_append_batch(self._h, len(slots), _p(slots, C.c_int32), _p(off, C.c_int64),
                                               _p(flat, C.c_int32), n_threads)

    def slot_len(self, slot: int) -> int:
        return int(self._lib.sfx_oracle_slot_len(self._h, slot))

    def slot_updates(self, slot: int) -> int:
        """Node updates made by the appends to `slot` since its last reset."""
        return int(self._lib.sfx_oracle_slot_updates(self._h, slot))

    def slot_text(self, slot: int) -> np.ndarray:
        out = np.empty(self.slot_len(slot), dtype=np.int32)
        self._lib.sfx_oracle_slot_text(self._h, slot, _p(out, C.c_int32))
        return out

    def count(self, tree: int, path) -> int:
        t = _i32(path)
        return int(self._lib.sfx_oracle_count(self._h, tree, _p(t, C.c_int32), t.size))

    def node_count(self, tree: int) -> int:
        return int(self._lib.sfx_oracle_node_count(self._h, tree))

    def dump(self, tree: int):
        """Pre-order (depth, parent, token, count) arrays, children by token."""
        n = self.node_count(tree)
        a = [np.empty(n, dtype=np.int32) for _ in range(4)]
        self._lib.sfx_oracle_dump(self._h, tree, n, *[_p(x, C.c_int32) for x in a])
        return tuple(a)

    def entropy(self, tree: int) -> float:
        return float(self._lib.sfx_oracle_entropy(self._h, tree))

    # ---- Algorithm 1 ---------------------------------------------------
    def budget(self, alpha: float, p: int, cap: int) -> int:
        return int(self._lib.sfx_oracle_budget(alpha, p, cap))

    def candidate(self, tree: int, context, p: int, budget: int, linear: bool = False):
        """(tokens, parents, D values, SCORE) of one (tree, p) candidate, or None."""
        ctx = _i32(context)
        cap = max(budget, 1)
        tok = np.empty(cap, dtype=np.int32)
        par = np.empty(cap, dtype=np.int32)
        dv = np.empty(cap, dtype=np.float64)
        sc = C.c_double(0.0)
        n = self._lib.sfx_oracle_candidate(self._h, tree, _p(ctx, C.c_int32), ctx.size, p, budget, int(linear),
                                           _p(tok, C.c_int32), _p(par, C.c_int32), _p(dv, C.c_double),
                                           C.byref(sc))
        if n < 0:
            return None
        return tok[:n].copy(), par[:n].copy(), dv[:n].copy(), sc.value

    def speculate(self, slots, P: int, alpha: float, max_spec: int, M: Optional[int] = None, flags: int = 0,
                  budget_override=None, n_threads: int = 1, tau: float = 0.0) -> dict:
        slots = _i32(slots)
        n = slots.size
        M = max_spec if M is None else M
        words = (M + 31) // 32
        r = {
            "n_draft": np.zeros(n, dtype=np.int32),
            "tokens": np.zeros((n, M), dtype=np.int32),
            "parents": np.zeros((n, M), dtype=np.int32),
            "positions": np.zeros((n, M), dtype=np.int32),
            "mask": np.zeros((n, M, words), dtype=np.uint32),
            "chosen_tree": np.zeros(n, dtype=np.int32),
            "chosen_p": np.zeros(n, dtype=np.int32),
            "score": np.zeros(n, dtype=np.float64),
            "visited": np.zeros((n, 3), dtype=np.int64),     # descents, added nodes, candidate trees
        }
        bo = None
        if budget_override is not None:
            bo_arr = _i32(budget_override)
            bo = _p(bo_arr, C.c_int32)
        self._lib.sfx_oracle_speculate(
            self._h, n, _p(slots, C.c_int32), P, float(alpha), max_spec, flags, M, bo,
            _p(r["n_draft"], C.c_int32), _p(r["tokens"], C.c_int32), _p(r["parents"], C.c_int32),
            _p(r["positions"], C.c_int32), _p(r["mask"], C.c_uint32), _p(r["chosen_tree"], C.c_int32),
            _p(r["chosen_p"], C.c_int32), _p(r["score"], C.c_double), _p(r["visited"], C.c_int64), n_threads,
            float(tau))
        return r
