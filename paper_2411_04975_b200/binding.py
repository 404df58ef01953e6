"""ctypes binding of libsuffixspec.so: argument marshalling only.

Tensors are torch CUDA tensors used as plain device buffers; the stream is
torch's current stream.  The module-level functions sd_build / sd_append /
sd_speculate / sd_free mirror the C entry points one to one; `SuffixStore`
wraps them with output allocation.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import torch

from . import build as _build

FLAG_GLOBAL_ONLY, FLAG_REQUEST_ONLY, FLAG_LINEAR = 1, 2, 4
STATUS_BAD_SLOT, STATUS_POOL_FULL, STATUS_GLOBAL_FULL, STATUS_BAD_TOKEN = 1, 2, 4, 8

EXPORTS = ["sd_build", "sd_build_requests", "sd_append", "sd_speculate", "sd_step", "sd_speculate_noalloc", "sd_query_counts",
           "sd_enumerate", "sd_slot_info", "sd_entropy", "sd_stats", "sd_free", "sd_strerror", "sd_debug_fail_alloc"]


class SuffixSpecError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {library().sd_strerror(code).decode()} ({code})")


class _BuildParams(C.Structure):
    _fields_ = [("vocab", C.c_int32), ("depth_cap", C.c_int32), ("max_requests", C.c_int32),
                ("max_req_tokens", C.c_int32), ("max_spec_cap", C.c_int32), ("global_extra_nodes", C.c_int64),
                ("slot_pool_nodes", C.c_int64)]


class _SpecParams(C.Structure):
    _fields_ = [("P", C.c_int32), ("alpha", C.c_double), ("max_spec", C.c_int32), ("flags", C.c_uint32),
                ("tau", C.c_double)]


class _Stats(C.Structure):
    _fields_ = [("global_nodes", C.c_int64), ("global_pool_used", C.c_int64), ("global_pool_cap", C.c_int64),
                ("global_tokens", C.c_int64), ("slot_pool_nodes", C.c_int64), ("device_bytes", C.c_int64),
                ("global_status", C.c_int32)]


_lib = None


def library() -> C.CDLL:
    """Load libsuffixspec.so (building it with nvcc if the sources are newer).
    Raises if it cannot be had: there is no fallback path."""
    global _lib
    if _lib is None:
        path = _build.LIB
        if not os.path.exists(path) or os.environ.get("SUFFIXSPEC_REBUILD"):
            path = _build.build()
        lib = C.CDLL(path)
        vp = C.c_void_p
        lib.sd_build.restype = C.c_int
        lib.sd_build.argtypes = [C.POINTER(_BuildParams), vp, vp, C.c_int32, vp, C.POINTER(vp)]
        lib.sd_build_requests.restype = C.c_int
        lib.sd_build_requests.argtypes = [vp, C.c_int32, vp, vp, vp, vp]
        lib.sd_append.restype = C.c_int
        lib.sd_append.argtypes = [vp, C.c_int32, vp, vp, vp, vp, vp]
        lib.sd_speculate.restype = C.c_int
        lib.sd_speculate.argtypes = [vp, C.c_int32, vp, C.POINTER(_SpecParams)] + [vp] * 11
        lib.sd_step.restype = C.c_int
        lib.sd_step.argtypes = [vp, C.c_int32, vp, vp, vp, C.POINTER(_SpecParams)] + [vp] * 11
        lib.sd_speculate_noalloc.restype = C.c_int
        lib.sd_speculate_noalloc.argtypes = lib.sd_speculate.argtypes
        lib.sd_query_counts.restype = C.c_int
        lib.sd_query_counts.argtypes = [vp, C.c_int32, vp, vp, vp, vp, vp]
        lib.sd_enumerate.restype = C.c_int
        lib.sd_enumerate.argtypes = [vp, C.c_int32, C.c_int64, vp, vp, vp, vp, C.POINTER(C.c_int64), vp]
        lib.sd_slot_info.restype = C.c_int
        lib.sd_slot_info.argtypes = [vp, C.c_int32, vp, vp, vp, vp, vp]
        lib.sd_entropy.restype = C.c_int
        lib.sd_entropy.argtypes = [vp, C.c_int32, C.POINTER(C.c_double), vp]
        lib.sd_stats.restype = C.c_int
        lib.sd_stats.argtypes = [vp, C.POINTER(_Stats), vp]
        lib.sd_free.restype = None
        lib.sd_free.argtypes = [vp]
        lib.sd_debug_fail_alloc.restype = None
        lib.sd_debug_fail_alloc.argtypes = [C.c_int64]
        lib.sd_strerror.restype = C.c_char_p
        lib.sd_strerror.argtypes = [C.c_int]
        _lib = lib
    return _lib


def _ptr(t: Optional[torch.Tensor], dtype: torch.dtype, name: str) -> Optional[int]:
    if t is None:
        return None
    # pinned host memory has a device address of its own (unified addressing): the kernels then
    # read or write it across the bus, with no copy before or after the call
    if not (t.is_cuda or t.is_pinned()) or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name}: expected a contiguous CUDA (or pinned host) tensor of {dtype}, "
                        f"got {t.dtype} on {t.device}")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


# ---- the C entry points, one to one ------------------------------------------------------
def sd_build(corpus: Optional[torch.Tensor], seq_offsets: Optional[torch.Tensor], *, vocab: int, depth_cap: int,
             max_requests: int, max_req_tokens: int, max_spec_cap: int, global_extra_nodes: int = -1,
             slot_pool_nodes: int = 0) -> int:
    """Returns the store handle (an integer address)."""
    p = _BuildParams(vocab, depth_cap, max_requests, max_req_tokens, max_spec_cap, global_extra_nodes,
                     slot_pool_nodes)
    n_seqs = 0 if seq_offsets is None else int(seq_offsets.numel()) - 1
    out = C.c_void_p()
    rc = library().sd_build(C.byref(p), _ptr(corpus, torch.int32, "corpus"),
                            _ptr(seq_offsets, torch.int64, "seq_offsets"), n_seqs, _stream(), C.byref(out))
    if rc != 0:
        raise SuffixSpecError(rc, "sd_build")
    return out.value


def sd_append(store: int, slots: torch.Tensor, offsets: torch.Tensor, tokens: torch.Tensor,
              reset: Optional[torch.Tensor] = None) -> None:
    rc = library().sd_append(store, int(slots.numel()), _ptr(slots, torch.int32, "slots"),
                             _ptr(offsets, torch.int64, "offsets"), _ptr(tokens, torch.int32, "tokens"),
                             _ptr(reset, torch.uint8, "reset"), _stream())
    if rc != 0:
        raise SuffixSpecError(rc, "sd_append")


def sd_speculate(store: int, slots: torch.Tensor, P: int, alpha: float, max_spec: int, flags: int,
                 budget_cap: Optional[torch.Tensor], out: Dict[str, torch.Tensor], tau: float = 0.0) -> None:
    prm = _SpecParams(P, alpha, max_spec, flags, tau)
    rc = library().sd_speculate(
        store, int(slots.numel()), _ptr(slots, torch.int32, "slots"), C.byref(prm),
        _ptr(budget_cap, torch.int32, "budget_cap"), _ptr(out["n_draft"], torch.int32, "n_draft"),
        _ptr(out["tokens"], torch.int32, "tokens"), _ptr(out["parents"], torch.int32, "parents"),
        _ptr(out["positions"], torch.int32, "positions"), _ptr(out["mask"], torch.int32, "mask"),
        _ptr(out["chosen_tree"], torch.int32, "chosen_tree"), _ptr(out["chosen_p"], torch.int32, "chosen_p"),
        _ptr(out["score"], torch.float64, "score"), _ptr(out["status"], torch.int32, "status"), _stream())
    if rc != 0:
        raise SuffixSpecError(rc, "sd_speculate")


def sd_speculate_noalloc(store: int, slots: torch.Tensor, P: int, alpha: float, max_spec: int, flags: int,
                         budget_cap: Optional[torch.Tensor], out: Dict[str, torch.Tensor], tau: float = 0.0) -> None:
    """sd_speculate for callers that may not allocate device memory: the scratch
    records live in a fixed array inside the library, so the batch is limited
    (n * 2 * depth_cap <= 4096 jobs) and calls on one device must not overlap.
    `out` must be preallocated by the caller; nothing is allocated here."""
    prm = _SpecParams(P, alpha, max_spec, flags, tau)
    rc = library().sd_speculate_noalloc(
        store, int(slots.numel()), _ptr(slots, torch.int32, "slots"), C.byref(prm),
        _ptr(budget_cap, torch.int32, "budget_cap"), _ptr(out["n_draft"], torch.int32, "n_draft"),
        _ptr(out["tokens"], torch.int32, "tokens"), _ptr(out["parents"], torch.int32, "parents"),
        _ptr(out["positions"], torch.int32, "positions"), _ptr(out["mask"], torch.int32, "mask"),
        _ptr(out["chosen_tree"], torch.int32, "chosen_tree"), _ptr(out["chosen_p"], torch.int32, "chosen_p"),
        _ptr(out["score"], torch.float64, "score"), _ptr(out["status"], torch.int32, "status"), _stream())
    if rc != 0:
        raise SuffixSpecError(rc, "sd_speculate_noalloc")


def sd_free(store: int) -> None:
    library().sd_free(store)


# ---- convenience wrapper ---------------------------------------------------------------------
class BoundStep:
    """One sd_step call with all of its arguments already converted (see SuffixStore.bind_step).
    Calling the object launches the step; `out` holds the output tensors it writes."""

    def __init__(self, store, slots, offsets, new_tokens, P, alpha, max_spec, flags, budget_cap, out, stream, tau=0.0):
        self.out = out
        self._keep = (store, slots, offsets, new_tokens, budget_cap)       # the buffers must outlive the calls
        self._prm = _SpecParams(P, alpha, max_spec, flags, tau)
        self._fn = library().sd_step
        self._args = (
            store._h, int(slots.numel()), _ptr(slots, torch.int32, "slots"), _ptr(offsets, torch.int64, "offsets"),
            _ptr(new_tokens, torch.int32, "new_tokens"), C.byref(self._prm), _ptr(budget_cap, torch.int32, "budget_cap"),
            _ptr(out["n_draft"], torch.int32, "n_draft"), _ptr(out["tokens"], torch.int32, "tokens"),
            _ptr(out["parents"], torch.int32, "parents"), _ptr(out["positions"], torch.int32, "positions"),
            _ptr(out["mask"], torch.int32, "mask"), _ptr(out["chosen_tree"], torch.int32, "chosen_tree"),
            _ptr(out["chosen_p"], torch.int32, "chosen_p"), _ptr(out["score"], torch.float64, "score"),
            _ptr(out["status"], torch.int32, "status"), stream)

    def __call__(self) -> Dict[str, torch.Tensor]:
        rc = self._fn(*self._args)
        if rc != 0:
            raise SuffixSpecError(rc, "sd_step")
        return self.out


class SuffixStore:
    """Global suffix tree + per-request trees on one GPU."""

    def __init__(self, corpus: Optional[torch.Tensor], seq_offsets: Optional[torch.Tensor], *, vocab: int,
                 depth_cap: int, max_requests: int, max_req_tokens: int, max_spec_cap: int,
                 global_extra_nodes: int = -1, slot_pool_nodes: int = 0):
        self.vocab, self.depth_cap, self.max_requests = vocab, depth_cap, max_requests
        self.max_req_tokens, self.max_spec_cap = max_req_tokens, max_spec_cap
        self.device = corpus.device if corpus is not None else torch.device("cuda", torch.cuda.current_device())
        self._h = sd_build(corpus, seq_offsets, vocab=vocab, depth_cap=depth_cap, max_requests=max_requests,
                           max_req_tokens=max_req_tokens, max_spec_cap=max_spec_cap,
                           global_extra_nodes=global_extra_nodes, slot_pool_nodes=slot_pool_nodes)

    @property
    def handle(self) -> int:
        return self._h

    def free(self) -> None:
        if self._h:
            sd_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass

    def append(self, slots: torch.Tensor, offsets: torch.Tensor, tokens: torch.Tensor,
               reset: Optional[torch.Tensor] = None) -> None:
        sd_append(self._h, slots, offsets, tokens, reset)

    def build_requests(self, slots, offsets, tokens: torch.Tensor) -> None:
        """Start new requests: `slots` and `offsets` are HOST sequences, `tokens` a CUDA tensor."""
        import numpy as np
        hs = np.ascontiguousarray(slots, dtype=np.int32)
        ho = np.ascontiguousarray(offsets, dtype=np.int64)
        rc = library().sd_build_requests(self._h, int(hs.size), hs.ctypes.data, ho.ctypes.data,
                                         _ptr(tokens, torch.int32, "tokens"), _stream())
        if rc != 0:
            raise SuffixSpecError(rc, "sd_build_requests")

    def alloc_outputs(self, n: int) -> Dict[str, torch.Tensor]:
        """Output tensors of sd_speculate for n requests.  They are views into ONE device
        buffer (returned under the key "packed"), so a caller that wants the drafts on the host
        needs a single device-to-host copy; `unpack_outputs` makes the same views on a host copy."""
        packed = torch.empty(self.packed_output_bytes(n), dtype=torch.uint8, device=self.device)
        return self.unpack_outputs(packed, n)

    def _output_layout(self, n: int):
        M = self.max_spec_cap
        words = (M + 31) // 32
        fields = [("score", torch.float64, (n,)), ("tokens", torch.int32, (n, M)), ("parents", torch.int32, (n, M)),
                  ("positions", torch.int32, (n, M)), ("mask", torch.int32, (n, M, words)),
                  ("n_draft", torch.int32, (n,)), ("chosen_tree", torch.int32, (n,)), ("chosen_p", torch.int32, (n,)),
                  ("status", torch.int32, (n,))]
        off, lay = 0, []
        for name, dt, shape in fields:
            size = torch.empty(0, dtype=dt).element_size()
            cnt = 1
            for d in shape:
                cnt *= d
            lay.append((name, dt, shape, off, cnt * size))
            off += (cnt * size + 15) // 16 * 16
        return lay, off

    def packed_output_bytes(self, n: int) -> int:
        return max(16, self._output_layout(n)[1])

    def unpack_outputs(self, packed: torch.Tensor, n: int) -> Dict[str, torch.Tensor]:
        lay, _ = self._output_layout(n)
        out = {"packed": packed}
        for name, dt, shape, off, nbytes in lay:
            out[name] = packed[off:off + nbytes].view(dt).view(shape)
        return out

    def speculate(self, slots: torch.Tensor, P: int, alpha: float, max_spec: int, flags: int = 0,
                  budget_cap: Optional[torch.Tensor] = None,
                  out: Optional[Dict[str, torch.Tensor]] = None, tau: float = 0.0) -> Dict[str, torch.Tensor]:
        """mask is returned as int32 words (same bits as the uint32 of the C ABI)."""
        if out is None:
            out = self.alloc_outputs(int(slots.numel()))
        sd_speculate(self._h, slots, P, alpha, max_spec, flags, budget_cap, out, tau)
        return out

    def step(self, slots: torch.Tensor, offsets: torch.Tensor, new_tokens: torch.Tensor, P: int, alpha: float,
             max_spec: int, flags: int = 0, budget_cap: Optional[torch.Tensor] = None,
             out: Optional[Dict[str, torch.Tensor]] = None, tau: float = 0.0) -> Dict[str, torch.Tensor]:
        """One decode step in one launch: append `new_tokens` (ragged by `offsets`) to the slots,
        then speculate.  Same result as append() followed by speculate()."""
        if out is None:
            out = self.alloc_outputs(int(slots.numel()))
        prm = _SpecParams(P, alpha, max_spec, flags, tau)
        rc = library().sd_step(
            self._h, int(slots.numel()), _ptr(slots, torch.int32, "slots"), _ptr(offsets, torch.int64, "offsets"),
            _ptr(new_tokens, torch.int32, "new_tokens"), C.byref(prm), _ptr(budget_cap, torch.int32, "budget_cap"),
            _ptr(out["n_draft"], torch.int32, "n_draft"), _ptr(out["tokens"], torch.int32, "tokens"),
            _ptr(out["parents"], torch.int32, "parents"), _ptr(out["positions"], torch.int32, "positions"),
            _ptr(out["mask"], torch.int32, "mask"), _ptr(out["chosen_tree"], torch.int32, "chosen_tree"),
            _ptr(out["chosen_p"], torch.int32, "chosen_p"), _ptr(out["score"], torch.float64, "score"),
            _ptr(out["status"], torch.int32, "status"), _stream())
        if rc != 0:
            raise SuffixSpecError(rc, "sd_step")
        return out

    def bind_step(self, slots: torch.Tensor, offsets: torch.Tensor, new_tokens: torch.Tensor, P: int, alpha: float,
                  max_spec: int, flags: int = 0, budget_cap: Optional[torch.Tensor] = None,
                  out: Optional[Dict[str, torch.Tensor]] = None, stream: Optional[int] = None,
                  tau: float = 0.0) -> "BoundStep":
        """step() with the argument marshalling done once.  A serving loop calls sd_step with the
        same buffers every step (it refills them in place: `new_tokens` is the whole token buffer,
        `offsets` says how much of it a step uses), so the returned object keeps the converted
        pointers and each call of it is just the C call.  `stream`: a cudaStream_t as an integer;
        default: the stream that is current now."""
        if out is None:
            out = self.alloc_outputs(int(slots.numel()))
        return BoundStep(self, slots, offsets, new_tokens, P, alpha, max_spec, flags, budget_cap, out,
                         _stream() if stream is None else stream, tau)

    def query_counts(self, tree: torch.Tensor, offsets: torch.Tensor, paths: torch.Tensor) -> torch.Tensor:
        n = int(tree.numel())
        counts = torch.empty(n, dtype=torch.int32, device=self.device)
        rc = library().sd_query_counts(self._h, n, _ptr(tree, torch.int32, "tree"),
                                       _ptr(offsets, torch.int64, "offsets"), _ptr(paths, torch.int32, "paths"),
                                       _ptr(counts, torch.int32, "counts"), _stream())
        if rc != 0:
            raise SuffixSpecError(rc, "sd_query_counts")
        return counts

    def enumerate(self, tree: int, max_nodes: int) -> Dict[str, torch.Tensor]:
        """All nodes of `tree` (-1: global) as records parent / token / count / depth (see sd_enumerate)."""
        o = {k: torch.empty(max(max_nodes, 1), dtype=torch.int32, device=self.device) for k in ("parent", "token", "count", "depth")}
        n = C.c_int64(0)
        rc = library().sd_enumerate(self._h, tree, max_nodes, o["parent"].data_ptr(), o["token"].data_ptr(),
                                    o["count"].data_ptr(), o["depth"].data_ptr(), C.byref(n), _stream())
        if rc != 0:
            raise SuffixSpecError(rc, "sd_enumerate")
        return {k: v[:n.value] for k, v in o.items()}

    def slot_info(self, slots: torch.Tensor):
        n = int(slots.numel())
        o = [torch.empty(n, dtype=torch.int32, device=self.device) for _ in range(3)]
        rc = library().sd_slot_info(self._h, n, _ptr(slots, torch.int32, "slots"), o[0].data_ptr(), o[1].data_ptr(),
                                    o[2].data_ptr(), _stream())
        if rc != 0:
            raise SuffixSpecError(rc, "sd_slot_info")
        return {"len": o[0], "nodes": o[1], "status": o[2]}

    def entropy(self, tree: int = -1) -> float:
        """Count-weighted mean entropy (bits) of the children distributions of `tree`."""
        h = C.c_double(0.0)
        rc = library().sd_entropy(self._h, tree, C.byref(h), _stream())
        if rc != 0:
            raise SuffixSpecError(rc, "sd_entropy")
        return h.value

    def stats(self) -> dict:
        st = _Stats()
        rc = library().sd_stats(self._h, C.byref(st), _stream())
        if rc != 0:
            raise SuffixSpecError(rc, "sd_stats")
        return {k: getattr(st, k) for k, _ in _Stats._fields_}
