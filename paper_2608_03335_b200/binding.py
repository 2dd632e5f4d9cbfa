"""ctypes binding of the C ABI in include/spade.h: argument marshalling only.

Every step of the path runs in the CUDA kernels of libspade_b200.so.  torch supplies device
memory and streams; nothing here computes.  If the library is missing the import of any
function below raises -- there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import torch

from .build import LIB, LIB_DEBUG, build_library

SPADE_TOPK, SPADE_TOPP, SPADE_SPARSITY, SPADE_POLICY_AS = 0, 1, 2, 3
ESTIMATORS = {"mean": 0, "dsa": 1, "dsa2": 2}       # spade_estimator_t
MODES = {"topk": SPADE_TOPK, "topp": SPADE_TOPP, "sparsity": SPADE_SPARSITY, "policy_as": SPADE_POLICY_AS}

ERRORS = {0: "SPADE_OK", -1: "SPADE_ERR_INVALID_ARG", -2: "SPADE_ERR_UNSUPPORTED", -3: "SPADE_ERR_WORKSPACE",
          -4: "SPADE_ERR_CUDA", -5: "SPADE_ERR_DEVICE_TIMEOUT", -6: "SPADE_ERR_ORDER", -7: "SPADE_ERR_DEBUG_CHECK"}


class SpadeError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"{ERRORS.get(code, code)}: {msg}")
        self.code = code


class Grid(C.Structure):
    _fields_ = [("T", C.c_int32), ("H", C.c_int32), ("W", C.c_int32), ("n_text", C.c_int32)]


class Blocking(C.Structure):
    _fields_ = [("bt", C.c_int32), ("bh", C.c_int32), ("bw", C.c_int32)]


class Budget(C.Structure):
    _fields_ = [("mode", C.c_int32), ("value", C.c_float), ("per_head", C.POINTER(C.c_float)), ("gain", C.c_float)]


class StaticMask(C.Structure):
    _fields_ = [("intra_threshold", C.c_float), ("window", C.c_int32), ("sink_tokens", C.c_int32)]


class Tables(C.Structure):
    _fields_ = [("BH", C.c_int32), ("C", C.c_int32), ("NBmax", C.c_int32), ("cap", C.c_int32),
                ("scheme", C.c_void_p), ("keep", C.c_void_p), ("as_", C.c_void_p), ("score", C.c_void_p),
                ("sics", C.c_void_p), ("NBvmax", C.c_int32), ("qsum", C.c_void_p), ("ksum", C.c_void_p),
                ("kv_idx", C.c_void_p), ("kv_cnt", C.c_void_p), ("head_order", C.c_void_p),
                ("group_count", C.c_void_p), ("item_start", C.c_void_p), ("cell_axis", C.c_void_p), ("status", C.c_void_p),
                ("minmax", C.c_void_p), ("block_scores", C.c_void_p), ("block_scores_ld", C.c_int32), ("cell_ld", C.c_int32)]


_lib = None


def lib():
    """Load libspade_b200.so (built in-tree by paper_2608_03335_b200.build); raise if absent."""
    global _lib
    if _lib is None:
        path = LIB
        if os.environ.get("SPADE_DEBUG") == "1":          # the checked build of the same kernels (see spade.h)
            path = build_library(debug=True)
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: build it with `python -m paper_2608_03335_b200.build` "
                               "(there is no CPU fallback)")
        L = C.CDLL(path)
        L.spade_last_error.restype = C.c_char_p
        L.spade_workspace_bytes.restype = C.c_size_t
        L.spade_workspace_bytes.argtypes = [C.c_void_p]
        L.spade_plan_create.argtypes = [C.POINTER(C.c_void_p), C.c_int32, C.c_int32, C.c_int32, C.POINTER(Grid),
                                        C.POINTER(Blocking), C.c_int32, C.POINTER(Budget), C.c_int32]
        L.spade_plan_destroy.argtypes = [C.c_void_p]
        vp = C.c_void_p
        ip = C.POINTER(C.c_int32)
        L.spade_plan.argtypes = [vp, vp, vp, vp, vp, ip]
        L.spade_summarize.argtypes = [vp, vp, vp, vp, vp]
        L.spade_select.argtypes = [vp, vp, vp]
        L.spade_attn.argtypes = [vp, vp, vp, vp, vp, vp, vp]
        L.spade_forward.argtypes = [vp, vp, vp, vp, vp, vp, vp, ip]
        L.spade_forward_host.argtypes = [vp] * 11 + [ip]
        L.spade_get_tables.argtypes = [vp, vp, C.POINTER(Tables)]
        L.spade_get_geometry.argtypes = [vp, C.c_int32, ip]
        L.spade_get_pair_table.argtypes = [vp, C.c_int32, ip, C.POINTER(C.c_uint32)]
        L.spade_status.argtypes = [vp, vp, vp]
        L.spade_launch_count.argtypes = [vp]
        L.spade_selftest_bounded_wait.argtypes = [vp, C.c_int32, vp]
        L.spade_plan_set_masks.argtypes = [vp, C.POINTER(StaticMask)]
        L.spade_plan_set_estimator.argtypes = [vp, C.c_int32]
        L.spade_aggregation_scores_noalloc.argtypes = [vp, vp, vp, vp, vp]
        _lib = L
    return _lib


def _check(rc: int):
    if rc != 0:
        raise SpadeError(rc, lib().spade_last_error().decode())


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _forced(forced: Optional[Sequence[int]]):
    if forced is None:
        return None
    return (C.c_int32 * len(forced))(*[int(x) for x in forced])


def spade_selftest_bounded_wait(limit_us: int = 2000, stream=None) -> Dict[str, int]:
    """Run the bounded-wait self-test; returns dict(gave_up, abort_flag, cycles)."""
    out = torch.zeros(4, dtype=torch.int32, device="cuda")
    _check(lib().spade_selftest_bounded_wait(_ptr(out), int(limit_us), _stream(stream)))
    torch.cuda.synchronize()
    o = out.cpu().tolist()
    return dict(gave_up=o[0], abort_flag=o[1], cycles=(o[2] & 0xffffffff) | ((o[3] & 0xffffffff) << 32))


class Plan:
    """Owns a spade_plan_t and its device workspace (a torch uint8 tensor)."""

    def __init__(self, B: int, heads: int, grid, n_text: int, candidates, mode: str, value: float,
                 per_head: Optional[Sequence[float]] = None, d: int = 128, device: int = 0,
                 intra_threshold: float = 0.0, window: int = -1, sink_tokens: int = 0, gain: float = 0.0,
                 estimator: str = "mean"):
        self.handle = C.c_void_p()
        self.B, self.heads, self.d = B, heads, d
        self.grid, self.n_text = tuple(grid), n_text
        self.candidates = [tuple(c) for c in candidates]
        self.N = grid[0] * grid[1] * grid[2] + n_text
        g = Grid(grid[0], grid[1], grid[2], n_text)
        cands = (Blocking * len(candidates))(*[Blocking(*c) for c in candidates])
        ph = None
        if per_head is not None:
            ph = (C.c_float * len(per_head))(*per_head)
        b = Budget(MODES[mode], float(value), C.cast(ph, C.POINTER(C.c_float)) if ph is not None else None, float(gain))
        _check(lib().spade_plan_create(C.byref(self.handle), B, heads, d, C.byref(g), cands, len(candidates),
                                       C.byref(b), device))
        if intra_threshold > 0 or window >= 0 or sink_tokens > 0:
            m = StaticMask(float(intra_threshold), int(window), int(sink_tokens))
            _check(lib().spade_plan_set_masks(self.handle, C.byref(m)))
        if estimator != "mean":
            if estimator not in ESTIMATORS:
                raise ValueError(f"estimator must be one of {sorted(ESTIMATORS)}")
            _check(lib().spade_plan_set_estimator(self.handle, ESTIMATORS[estimator]))
        self.estimator = estimator
        self.device = torch.device("cuda", device)
        self.ws_bytes = int(lib().spade_workspace_bytes(self.handle))
        self.ws = torch.empty(self.ws_bytes + 256, dtype=torch.uint8, device=self.device)
        off = (-self.ws.data_ptr()) % 256
        self._ws_ptr = C.c_void_p(self.ws.data_ptr() + off)

    def close(self):
        if self.handle:
            lib().spade_plan_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the four stages (same names as the C ABI) ------------------------------------------
    def spade_plan(self, Q, K, forced_scheme=None, stream=None):
        _check(lib().spade_plan(self.handle, _ptr(Q), _ptr(K), self._ws_ptr, _stream(stream), _forced(forced_scheme)))

    def spade_summarize(self, Q, K, stream=None):
        _check(lib().spade_summarize(self.handle, _ptr(Q), _ptr(K), self._ws_ptr, _stream(stream)))

    def spade_select(self, stream=None):
        _check(lib().spade_select(self.handle, self._ws_ptr, _stream(stream)))

    def spade_attn(self, Q, K, V, O, stream=None):
        _check(lib().spade_attn(self.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(O), self._ws_ptr, _stream(stream)))

    def spade_forward(self, Q, K, V, O, forced_scheme=None, stream=None):
        _check(lib().spade_forward(self.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(O), self._ws_ptr, _stream(stream),
                                   _forced(forced_scheme)))

    def spade_forward_host(self, hQ, hK, hV, hO, dQ, dK, dV, dO, forced_scheme=None, stream=None):
        _check(lib().spade_forward_host(self.handle, _ptr(hQ), _ptr(hK), _ptr(hV), _ptr(hO), _ptr(dQ), _ptr(dK),
                                        _ptr(dV), _ptr(dO), self._ws_ptr, _stream(stream), _forced(forced_scheme)))

    def spade_aggregation_scores_noalloc(self, Q, K, as_out, stream=None):
        """AS(Q|c), AS(K|c) per head and candidate into `as_out` (float32 [B*heads, n_cands, 2]) without
        touching the workspace or allocating: for callers that cannot get device memory (see spade.h)."""
        _check(lib().spade_aggregation_scores_noalloc(self.handle, _ptr(Q), _ptr(K), _ptr(as_out), _stream(stream)))

    def spade_status(self, stream=None):
        _check(lib().spade_status(self.handle, self._ws_ptr, _stream(stream)))

    def launch_count(self) -> int:
        return int(lib().spade_launch_count(self.handle))

    def geometry(self, cand: int) -> Dict[str, int]:
        out = (C.c_int32 * 6)()
        _check(lib().spade_get_geometry(self.handle, cand, out))
        return dict(nbt=out[0], nbh=out[1], nbw=out[2], NBv=out[3], NBt=out[4], BS=out[5], NB=out[3] + out[4])

    def pair_table(self, cand: int):
        """Tiles of a 64-token candidate: (tile_cell[tiles], pairs[tiles][3]) as int64 tensors on the host;
        pairs[t][a] = qb0 | qb1 << 16 when the tile's cell pairs along axis a (qb1 = 0xffff: a lone block).
        None for a 128-token candidate."""
        n = int(lib().spade_get_pair_table(self.handle, cand, None, None))
        if n < 0:
            _check(n)
        if n == 0:
            return None
        tc = (C.c_int32 * n)()
        pr = (C.c_uint32 * (3 * n))()
        _check(min(0, int(lib().spade_get_pair_table(self.handle, cand, tc, pr))))
        return (torch.tensor(list(tc), dtype=torch.int64), torch.tensor(list(pr), dtype=torch.int64).view(n, 3))

    # ---- tables (device views into the workspace) ------------------------------------------
    def tables(self) -> Dict[str, torch.Tensor]:
        t = Tables()
        _check(lib().spade_get_tables(self.handle, self._ws_ptr, C.byref(t)))
        base = self.ws.data_ptr()

        def view(ptr, dtype, shape):
            n = 1
            for s in shape:
                n *= s
            off = ptr - base
            el = torch.empty(0, dtype=dtype).element_size()
            return self.ws[off:off + n * el].view(dtype).view(*shape)

        BH, Cn, NB, cap, NBv = t.BH, t.C, t.NBmax, t.cap, t.NBvmax
        i32, f32 = torch.int32, torch.float32
        extra = {}
        if t.minmax:
            extra["minmax"] = view(t.minmax, f32, (4, BH, 128, t.block_scores_ld))
        return dict(block_scores=view(t.block_scores, f32, (BH, NBv, t.block_scores_ld)), **extra,
                    scheme=view(t.scheme, i32, (BH,)), keep=view(t.keep, i32, (BH,)),
                    as_=view(t.as_, f32, (BH, Cn, 2)), score=view(t.score, f32, (BH, Cn)),
                    sics=view(t.sics, f32, (BH, Cn, 2, NBv)), qsum=view(t.qsum, f32, (BH, NB, 128)),
                    ksum=view(t.ksum, f32, (BH, NB, 128)), kv_idx=view(t.kv_idx, i32, (BH, NB, cap)),
                    kv_cnt=view(t.kv_cnt, i32, (BH, NB)), head_order=view(t.head_order, i32, (BH,)),
                    group_count=view(t.group_count, i32, (8,)), item_start=view(t.item_start, i32, (BH + 1,)),
                    cell_axis=view(t.cell_axis, torch.uint8, (BH, t.cell_ld)),
                    status=view(t.status, i32, (4,)), cap=cap, NBmax=NB)
