"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE -- never a product path).

Only tests, the smoke check and the bench's CPU-baseline leg import this module.  It builds
`libspade_oracle.so` from `spade_oracle.cpp` with g++ on first use and exposes the oracle's
steps with numpy arrays.  Tensors are passed per head as [N, d] arrays, either raw bf16 bits
(uint16) or float64.  Nothing here imports the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spade_oracle.cpp")
_LIB = os.path.join(_HERE, "libspade_oracle.so")
_SANITIZE = os.environ.get("SPADE_ORACLE_SANITIZE") == "1"     # AddressSanitizer + UBSan build (run under LD_PRELOAD=libasan)
if _SANITIZE:
    _LIB = os.path.join(_HERE, "libspade_oracle_san.so")
_lib = None

_I = C.POINTER(C.c_int)
_D = C.POINTER(C.c_double)


def build(force: bool = False) -> str:
    """Compile the oracle (g++ -O2, no fast-math: fp64 with the order the source states)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        san = ["-fsanitize=address,undefined", "-fno-sanitize-recover=undefined", "-g", "-O1"] if _SANITIZE else ["-O2"]
        subprocess.check_call(["g++"] + san + ["-std=c++17", "-fPIC", "-shared", "-pthread",
                               "-ffp-contract=off", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.so_aggregate.restype = C.c_double
        _lib.so_norm_z.restype = C.c_double
        _lib.so_sparsity.restype = C.c_double
    return _lib


def _ip(a):
    return a.ctypes.data_as(_I)


def _dp(a):
    return a.ctypes.data_as(_D)


def _i32(seq):
    return np.ascontiguousarray(np.asarray(seq, dtype=np.int32))


def _tensor(x) -> Tuple[np.ndarray, int]:
    x = np.ascontiguousarray(x)
    if x.dtype == np.uint16:
        return x, 0
    if x.dtype == np.float64:
        return x, 1
    raise TypeError(f"oracle tensors are uint16 (bf16 bits) or float64, got {x.dtype}")


def _grid(grid, n_text=0):
    return _i32(list(grid) + [n_text])


# ---------------------------------------------------------------- geometry (Sec. 3.1, Fig. 3)
def geometry(grid, n_text, blk) -> Dict[str, int]:
    out = np.zeros(6, np.int32)
    rc = lib().so_geometry(_ip(_grid(grid, n_text)), _ip(_i32(blk)), _ip(out))
    if rc:
        raise ValueError("bad grid / blocking")
    return dict(nbt=int(out[0]), nbh=int(out[1]), nbw=int(out[2]), NBv=int(out[3]), NBt=int(out[4]), BS=int(out[5]),
                NB=int(out[3] + out[4]))


def block_tokens(grid, n_text, blk, block_id) -> np.ndarray:
    g = geometry(grid, n_text, blk)
    tok = np.zeros(g["BS"], np.int32)
    n = lib().so_block_tokens(_ip(_grid(grid, n_text)), _ip(_i32(blk)), int(block_id), _ip(tok))
    if n < 0:
        raise IndexError(block_id)
    return tok[:n].copy()


def block_sizes(grid, n_text, blk) -> np.ndarray:
    g = geometry(grid, n_text, blk)
    out = np.zeros(g["NB"], np.int32)
    lib().so_block_sizes(_ip(_grid(grid, n_text)), _ip(_i32(blk)), _ip(out))
    return out


# ---------------------------------------------------------------- SICS / AS (Eq. 3-5, Alg. 1)
def sics_blocks(x, grid, n_text, blk, threads=0) -> np.ndarray:
    """Per-video-block SICS of one head's [N, d] tensor."""
    x, dt = _tensor(x)
    g = geometry(grid, n_text, blk)
    out = np.zeros(g["NBv"], np.float64)
    lib().so_sics_blocks(x.ctypes.data_as(C.c_void_p), dt, x.shape[-1], _ip(_grid(grid, n_text)), _ip(_i32(blk)),
                         _dp(out), threads)
    return out


def aggregation_score(x, grid, n_text, blk, threads=0) -> float:
    s = sics_blocks(x, grid, n_text, blk, threads)
    return float(lib().so_aggregate(_dp(s), len(s)))


def norm_z(grid, n_text, blk) -> float:
    return float(lib().so_norm_z(_ip(_grid(grid, n_text)), _ip(_i32(blk))))


def choose_scheme(as_q: Sequence[float], as_k: Sequence[float], z: Sequence[float]) -> Tuple[int, np.ndarray]:
    aq = np.ascontiguousarray(as_q, np.float64)
    ak = np.ascontiguousarray(as_k, np.float64)
    zz = np.ascontiguousarray(z, np.float64)
    score = np.zeros(len(aq), np.float64)
    c = lib().so_choose(_dp(aq), _dp(ak), _dp(zz), len(aq), _dp(score))
    return int(c), score


# ---------------------------------------------------------------- summaries, estimator, select
def summaries(x, grid, n_text, blk, threads=0) -> np.ndarray:
    x, dt = _tensor(x)
    g = geometry(grid, n_text, blk)
    out = np.zeros((g["NB"], x.shape[-1]), np.float64)
    lib().so_summaries(x.ctypes.data_as(C.c_void_p), dt, x.shape[-1], _ip(_grid(grid, n_text)), _ip(_i32(blk)),
                       _dp(out), threads)
    return out


def block_scores(qs: np.ndarray, ks: np.ndarray, nbv: int, threads=0) -> Tuple[np.ndarray, np.ndarray]:
    qs = np.ascontiguousarray(qs[:nbv], np.float64)
    ks = np.ascontiguousarray(ks[:nbv], np.float64)
    S = np.zeros((nbv, nbv), np.float64)
    P = np.zeros((nbv, nbv), np.float64)
    lib().so_block_scores(_dp(qs), _dp(ks), nbv, qs.shape[1], _dp(S), _dp(P), threads)
    return S, P


def summaries_minmax(x, grid, n_text, blk, threads=0) -> Tuple[np.ndarray, np.ndarray]:
    """Channel-wise max and min of every block (Sec. 3.1, Summarizer Expression)."""
    x, dt = _tensor(x)
    g = geometry(grid, n_text, blk)
    mx = np.zeros((g["NB"], x.shape[-1]), np.float64)
    mn = np.zeros((g["NB"], x.shape[-1]), np.float64)
    lib().so_summaries_minmax(x.ctypes.data_as(C.c_void_p), dt, x.shape[-1], _ip(_grid(grid, n_text)), _ip(_i32(blk)),
                              _dp(mx), _dp(mn), threads)
    return mx, mn


ESTIMATORS = {"mean": 0, "dsa": 1, "dsa2": 2}


def block_scores_dsa(qmax, qmin, kmax, kmin, nbv: int, variant: str, threads=0) -> Tuple[np.ndarray, np.ndarray]:
    """Max/min-summary estimators (Fig. 4a "dsa", Fig. 4b "dsa2") on the video blocks."""
    a = [np.ascontiguousarray(t[:nbv], np.float64) for t in (qmax, qmin, kmax, kmin)]
    S = np.zeros((nbv, nbv), np.float64)
    P = np.zeros((nbv, nbv), np.float64)
    rc = lib().so_block_scores_dsa(_dp(a[0]), _dp(a[1]), _dp(a[2]), _dp(a[3]), nbv, a[0].shape[1], ESTIMATORS[variant],
                                   _dp(S), _dp(P), threads)
    if rc:
        raise ValueError("variant must be 'dsa' or 'dsa2'")
    return S, P


def keep_count(sparsity: float, nkb: int) -> int:
    return int(lib().so_keep_count(C.c_double(sparsity), nkb))


def select(S, P, nbv, nbt, mode: str, value: float, cap: Optional[int] = None, threads=0):
    """mode 'topk' | 'topp' | 'sparsity' -> (kv_idx [NB, cap] int32 (-1 padded), kv_cnt [NB])."""
    nb = nbv + nbt
    cap = nb if cap is None else cap
    if mode == "sparsity":
        mode, value = "topk", keep_count(value, nbv)
    m = {"topk": 0, "topp": 1}[mode]
    S = np.ascontiguousarray(S, np.float64)
    P = np.ascontiguousarray(P, np.float64)
    idx = np.full((nb, cap), -1, np.int32)
    cnt = np.zeros(nb, np.int32)
    rc = lib().so_select(_dp(S), _dp(P), nbv, nbt, m, C.c_double(float(value)), _ip(idx), _ip(cnt), cap, threads)
    if rc:
        raise ValueError("list capacity too small")
    return idx, cnt


def policy_keep_counts(selected_scores, nkb, mean_sparsity: float, gain: float):
    """Example policy function (Sec. 3.1 / 4.4: the keep budget is negatively correlated with the head's
    Selected Aggregation Score).  Reading: with a_h the selected normalised score and a_bar its mean over
    heads, head h keeps the fraction f_h = clamp((1 - s) * (1 - gain * (a_h - a_bar) / a_bar), 1/NKB_h, 1)
    of its video KV blocks: k_h = clamp(ceil(f_h * NKB_h - 1e-9), 1, NKB_h).  Returns (k, f)."""
    a = np.asarray(selected_scores, np.float64)
    nkb = np.asarray(nkb, np.int64)
    abar = float(a.sum() / len(a))
    f = (1.0 - mean_sparsity) * (1.0 - gain * (a - abar) / abar)
    f = np.minimum(np.maximum(f, 1.0 / nkb), 1.0)
    k = np.ceil(f * nkb - 1e-9).astype(np.int64)
    return np.clip(k, 1, nkb), f


def apply_static(grid, n_text, blk, kv_idx, kv_cnt, sics_q, sics_k, intra_threshold=0.0, window=-1, sink_tokens=0):
    """Union of the dynamic lists with the intra-block, local-window and attention-sink masks (in place)."""
    kv_idx = np.ascontiguousarray(kv_idx, np.int32)
    kv_cnt = np.ascontiguousarray(kv_cnt, np.int32)
    sq = np.ascontiguousarray(sics_q, np.float64)
    sk = np.ascontiguousarray(sics_k, np.float64)
    rc = lib().so_apply_static(_ip(_grid(grid, n_text)), _ip(_i32(blk)), _ip(kv_idx), _ip(kv_cnt), kv_idx.shape[1],
                               _dp(sq), _dp(sk), C.c_double(float(intra_threshold)), int(window), int(sink_tokens))
    if rc:
        raise ValueError("list capacity too small")
    return kv_idx, kv_cnt


# ---------------------------------------------------------------- attention (Eq. 2)
def attention_blocks(Q, K, V, grid, n_text, blk, q_blocks, kv_idx, kv_cnt, threads=0):
    """Block-sparse attention of the query blocks `q_blocks` of one head.

    Returns (out [n_q, BS, d] float64, tok [n_q, BS] int32 with -1 for absent rows)."""
    Q, dt = _tensor(Q)
    K, dk = _tensor(K)
    V, dv = _tensor(V)
    assert dt == dk == dv
    g = geometry(grid, n_text, blk)
    qb = _i32(q_blocks)
    kv_idx = np.ascontiguousarray(kv_idx, np.int32)
    kv_cnt = np.ascontiguousarray(kv_cnt, np.int32)
    d = Q.shape[-1]
    out = np.zeros((len(qb), g["BS"], d), np.float64)
    tok = np.zeros((len(qb), g["BS"]), np.int32)
    rc = lib().so_attention_blocks(Q.ctypes.data_as(C.c_void_p), K.ctypes.data_as(C.c_void_p),
                                   V.ctypes.data_as(C.c_void_p), dt, d, _ip(_grid(grid, n_text)), _ip(_i32(blk)),
                                   _ip(qb), len(qb), _ip(kv_idx), _ip(kv_cnt), kv_idx.shape[1], _dp(out), _ip(tok),
                                   threads)
    if rc:
        raise ValueError("bad block list")
    return out, tok


def sparsity(grid, n_text, blk, kv_idx, kv_cnt) -> float:
    kv_idx = np.ascontiguousarray(kv_idx, np.int32)
    kv_cnt = np.ascontiguousarray(kv_cnt, np.int32)
    return float(lib().so_sparsity(_ip(_grid(grid, n_text)), _ip(_i32(blk)), _ip(kv_idx), _ip(kv_cnt),
                                   kv_idx.shape[1]))


# ---------------------------------------------------------------- the selection pipeline, per head
def plan_head(q, k, grid, n_text, cands, forced: Optional[int] = None, threads=0):
    """Scheme generation for one head: AS(Q|c), AS(K|c) for every candidate, normalised score, argmax."""
    asq = [aggregation_score(q, grid, n_text, c, threads) for c in cands]
    ask = [aggregation_score(k, grid, n_text, c, threads) for c in cands]
    z = [norm_z(grid, n_text, c) for c in cands]
    best, score = choose_scheme(asq, ask, z)
    return dict(as_q=np.array(asq), as_k=np.array(ask), z=np.array(z), score=score,
                scheme=best if forced is None else int(forced))


def select_head(q, k, grid, n_text, blk, mode, value, threads=0, static=None, estimator="mean"):
    """Summaries -> estimator -> index search (-> union with the static masks) for one head under `blk`.

    static: optional dict(intra_threshold=, window=, sink_tokens=); estimator: "mean", "dsa" or "dsa2"."""
    g = geometry(grid, n_text, blk)
    qs = summaries(q, grid, n_text, blk, threads)
    ks = summaries(k, grid, n_text, blk, threads)
    if estimator == "mean":
        S, P = block_scores(qs, ks, g["NBv"], threads)
    else:
        qmx, qmn = summaries_minmax(q, grid, n_text, blk, threads)
        kmx, kmn = summaries_minmax(k, grid, n_text, blk, threads)
        S, P = block_scores_dsa(qmx, qmn, kmx, kmn, g["NBv"], estimator, threads)
    idx, cnt = select(S, P, g["NBv"], g["NBt"], mode, value, threads=threads)
    out = dict(qs=qs, ks=ks, S=S, P=P, kv_idx=idx, kv_cnt=cnt, geo=g, dyn_idx=idx.copy(), dyn_cnt=cnt.copy())
    if static:
        sq = sics_blocks(q, grid, n_text, blk, threads)
        sk = sics_blocks(k, grid, n_text, blk, threads)
        apply_static(grid, n_text, blk, idx, cnt, sq, sk, **static)
        out.update(sics_q=sq, sics_k=sk)
    return out
