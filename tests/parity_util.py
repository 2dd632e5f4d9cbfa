"""Shared machinery of the GPU parity tests: run the CUDA path stage by stage through the C ABI
and compare each stage with the CPU oracle on the same bytes.

Tolerances (also written where they are used):
  * SICS / AS / summaries: fp32 accumulation of <= 128 bf16 rows against fp64 -> rtol 2e-5.
  * scheme choice: exact, unless the two best normalised scores differ by < 1e-5 relative
    (counted, then the GPU's choice is forced into the oracle).
  * index lists: exact as sets, except blocks whose block score is within 1e-4 (logit units,
    i.e. 1e-4 relative on the probability) of the cut; Top-P prefix lengths may differ only
    when the oracle's running mass at the cut is within 1e-4*p of p.  Excused blocks are counted.
  * block scores of the mean estimator (Sec. 3.1, Fig. 4c), element by element, against the bound
    M = max_ij sum_c |Q'_ic K'_jc| / sqrt(d): within 3e-6 * M of the oracle's estimator fed the GPU's own
    fp32 summaries (the kernel's arithmetic alone: fp32 accumulation in the tensor core, which does not round to nearest, plus the dropped 2^-22 term), and
    within 6e-6 * M of the oracle's own chain (the fp32 summaries add their rounding).  A single TF32
    product cuts both operands to 10 mantissa bits, an error of about 2^-10 per term that does not
    average out below 4e-5 * M over 128 channels: it fails both.
  * attention, given the GPU's own lists: max-abs 2e-2 and relative Frobenius 5e-3.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from oracle import spade_oracle as so
from paper_2608_03335_b200 import binding
from paper_2608_03335_b200.workloads import Workload, bf16_bits, make_qkv

SCORE_REL = 6e-6          # of the largest sum of product magnitudes of the head; whole chain against the oracle
SCORE_REL_KERNEL = 3e-6   # same, the estimator alone (oracle fed the GPU's summaries)
ATTN_MAX_ABS = 2e-2
ATTN_REL_FRO = 5e-3
CUT_MARGIN = 1e-4
SCHEME_TIE = 1e-5


@dataclasses.dataclass
class Report:
    scheme_ties: int = 0
    near_cut_blocks: int = 0
    rows_checked: int = 0
    attn_blocks: int = 0
    attn_max_abs: float = 0.0
    attn_rel_fro: float = 0.0
    sparsity: float = 0.0
    score_err_rel: float = 0.0
    score_err_kernel: float = 0.0


def make_plan(w: Workload, per_head=None, static=None, estimator="mean") -> binding.Plan:
    return binding.Plan(w.batch, w.heads, w.grid, w.n_text, w.candidates, w.mode, w.value, per_head=per_head,
                        estimator=estimator, **(static or {}))


def oracle_value(w: Workload) -> float:
    """The budget value as the C ABI sees it (a float32)."""
    return float(np.float32(w.value))


def check_plan(w: Workload, plan: binding.Plan, qb, kb, rep: Report, forced=None):
    """Stage 1 against the oracle; returns the per-head scheme the GPU chose."""
    t = plan.tables()
    scheme = t["scheme"].cpu().numpy()
    BH = w.batch * w.heads
    if forced is not None:
        assert scheme.tolist() == list(forced)
        return scheme
    sics = t["sics"].cpu().numpy()
    as_ = t["as_"].cpu().numpy()
    score = t["score"].cpu().numpy()
    for bh in range(BH):
        p = so.plan_head(qb[bh], kb[bh], w.grid, w.n_text, w.candidates)
        for c, blk in enumerate(w.candidates):
            nbv = so.geometry(w.grid, w.n_text, blk)["NBv"]
            ref_q = so.sics_blocks(qb[bh], w.grid, w.n_text, blk)
            ref_k = so.sics_blocks(kb[bh], w.grid, w.n_text, blk)
            np.testing.assert_allclose(sics[bh, c, 0, :nbv], ref_q, rtol=2e-5, atol=1e-4)
            np.testing.assert_allclose(sics[bh, c, 1, :nbv], ref_k, rtol=2e-5, atol=1e-4)
        np.testing.assert_allclose(as_[bh, :, 0], p["as_q"], rtol=2e-5)
        np.testing.assert_allclose(as_[bh, :, 1], p["as_k"], rtol=2e-5)
        np.testing.assert_allclose(score[bh], p["score"], rtol=2e-5)
        if scheme[bh] != p["scheme"]:
            s = np.sort(p["score"])[::-1]
            assert (s[0] - p["score"][scheme[bh]]) / abs(s[0]) < SCHEME_TIE, \
                f"head {bh}: GPU scheme {scheme[bh]} vs oracle {p['scheme']} scores {p['score']}"
            rep.scheme_ties += 1
    return scheme


def check_summaries(w: Workload, plan: binding.Plan, qb, kb, scheme):
    t = plan.tables()
    qs, ks = t["qsum"].cpu().numpy(), t["ksum"].cpu().numpy()
    for bh in range(w.batch * w.heads):
        blk = w.candidates[scheme[bh]]
        rq = so.summaries(qb[bh], w.grid, w.n_text, blk)
        rk = so.summaries(kb[bh], w.grid, w.n_text, blk)
        np.testing.assert_allclose(qs[bh, :len(rq)], rq, rtol=2e-5, atol=2e-6)
        np.testing.assert_allclose(ks[bh, :len(rk)], rk, rtol=2e-5, atol=2e-6)


def _check_row_topk(S, kept, ref, k, rep: Report, margin=CUT_MARGIN):
    if kept == ref:
        return
    order = np.sort(S)[::-1]
    cut_hi, cut_lo = order[k - 1], order[k] if k < len(order) else order[k - 1]
    for j in set(kept) ^ set(ref):
        assert min(abs(S[j] - cut_hi), abs(S[j] - cut_lo)) < margin, \
            f"block {j} differs with score {S[j]} vs cut [{cut_lo}, {cut_hi}]"
        rep.near_cut_blocks += 1


def _near_topp_cut(S, run, pos, j, cut, p, margin):
    """A block may differ between the two sides when its score is at the cut, or when the oracle's running
    mass just before or just after it is within 1e-4 * p of p (there the prefix length is decided by rounding)."""
    r = pos[j]
    before = run[r - 1] if r > 0 else 0.0
    return abs(S[j] - cut) < margin or abs(before - p) <= CUT_MARGIN * p or abs(run[r] - p) <= CUT_MARGIN * p


def _check_row_topp(S, P, kept, ref, p, rep: Report, margin=CUT_MARGIN):
    if kept == ref:
        return
    order = sorted(range(len(S)), key=lambda j: (-S[j], j))
    m = len(kept)
    run = np.cumsum(P[order])
    assert run[m - 1] >= p * (1 - CUT_MARGIN), f"kept mass {run[m - 1]} < p"
    if m > 1:
        assert run[m - 2] < p * (1 + CUT_MARGIN), f"prefix not minimal: mass without last {run[m - 2]}"
    cut = S[order[m - 1]]
    pos = {j: r for r, j in enumerate(order)}
    for j in set(kept) ^ set(order[:m]):
        assert _near_topp_cut(S, run, pos, j, cut, p, margin), f"block {j} (score {S[j]}) is not near the cut {cut}"
    rep.near_cut_blocks += len(set(kept) ^ set(ref))


def check_minmax(w: Workload, plan: binding.Plan, qb, kb, scheme, estimator: str):
    """Max / min summaries (bit-exact: the values are bf16) and the estimator's scores against the oracle."""
    t = plan.tables()
    mm = t["minmax"].cpu().numpy()
    S_gpu = t["block_scores"].cpu().numpy()
    for bh in range(w.batch * w.heads):
        blk = w.candidates[scheme[bh]]
        nbv = so.geometry(w.grid, w.n_text, blk)["NBv"]
        qmx, qmn = so.summaries_minmax(qb[bh], w.grid, w.n_text, blk)
        kmx, kmn = so.summaries_minmax(kb[bh], w.grid, w.n_text, blk)
        # stored channel-major; every plane is one or two exact fp32 operations on bf16 values
        f = [x[:nbv].astype(np.float32) for x in (qmx, qmn, kmx, kmn)]
        half = np.float32(0.5)
        planes = (half * (f[0] + f[1]) if estimator == "dsa" else f[0], f[1], half * (f[2] + f[3]), half * (f[2] - f[3]))
        for plane, ref in enumerate(planes):
            np.testing.assert_array_equal(mm[plane, bh, :, :nbv], ref.T)
        S, _ = so.block_scores_dsa(qmx, qmn, kmx, kmn, nbv, estimator)
        # fp32 sum of 128 products against fp64: the error scales with the sum of the magnitudes
        tol = 2e-6 * float(np.abs(S).max() + 1.0) * 8
        np.testing.assert_allclose(S_gpu[bh, :nbv, :nbv], S, atol=max(tol, 1e-5), rtol=0)


def check_select(w: Workload, plan: binding.Plan, qb, kb, scheme, rep: Report, rows_per_head: Optional[int] = None,
                 rng=None, static=None, estimator="mean"):
    """Stage 3 against the oracle (which runs summaries -> estimator -> search itself, in fp64)."""
    t = plan.tables()
    kv_idx, kv_cnt = t["kv_idx"].cpu().numpy(), t["kv_cnt"].cpu().numpy()
    keep = t["keep"].cpu().numpy()
    value = oracle_value(w)
    spars = []
    for bh in range(w.batch * w.heads):
        blk = w.candidates[scheme[bh]]
        g = so.geometry(w.grid, w.n_text, blk)
        sel = so.select_head(qb[bh], kb[bh], w.grid, w.n_text, blk, w.mode, value, static=static, estimator=estimator)
        nbv, nbt, nb = g["NBv"], g["NBt"], g["NB"]
        if estimator == "mean":
            # the estimator's table itself, element by element (Sec. 3.1, Fig. 4c)
            S_gpu = t["block_scores"][bh, :nbv, :nbv].cpu().numpy()
            bound = float((np.abs(sel["qs"][:nbv]) @ np.abs(sel["ks"][:nbv]).T).max()) / np.sqrt(w.d)
            err = float(np.abs(S_gpu - sel["S"][:nbv, :nbv]).max())
            assert err <= SCORE_REL * bound, f"head {bh}: block scores off by {err:.3e} (bound {SCORE_REL * bound:.3e})"
            S_own, _ = so.block_scores(t["qsum"][bh, :nb].cpu().numpy().astype(np.float64),
                                       t["ksum"][bh, :nb].cpu().numpy().astype(np.float64), nbv)
            err_k = float(np.abs(S_gpu - S_own[:nbv, :nbv]).max())
            assert err_k <= SCORE_REL_KERNEL * bound, f"head {bh}: estimator kernel off by {err_k:.3e} (bound {SCORE_REL_KERNEL * bound:.3e})"
            rep.score_err_rel = max(rep.score_err_rel, err / bound)
            rep.score_err_kernel = max(rep.score_err_kernel, err_k / bound)
        # near-cut margin: 1e-4 on the mean estimator's O(1) scores; the max/min estimators add 128 products
        # of one sign pattern in fp32, so their rounding error grows with the score's magnitude
        margin = CUT_MARGIN if estimator == "mean" else max(CUT_MARGIN, 1e-5 * float(np.abs(sel["S"]).max()))
        if static and static.get("intra_threshold", 0) > 0:
            # the threshold must not sit on a block's value (fp32 vs fp64 would then decide differently)
            sizes = so.block_sizes(w.grid, w.n_text, blk)[:nbv].astype(np.float64) ** 2
            for sc in (sel["sics_q"], sel["sics_k"]):
                assert np.abs(sc / sizes - static["intra_threshold"]).min() > 1e-5, "pick another threshold"
        if w.mode != "topp":
            k = int(value) if w.mode == "topk" else so.keep_count(value, nbv)
            k = max(1, min(k, nbv))
            assert keep[bh] == k
        rows = range(nb)
        if rows_per_head is not None and rows_per_head < nb:
            rows = sorted(set([0, nbv - 1, nb - 1] + list(rng.choice(nb, rows_per_head, replace=False))))
        for i in rows:
            cnt = int(kv_cnt[bh, i])
            kept = kv_idx[bh, i, :cnt].tolist()
            ref = sel["kv_idx"][i, :sel["kv_cnt"][i]].tolist()
            assert kept == sorted(set(kept)) and all(0 <= j < nb for j in kept), "list not ascending / in range"
            if i >= nbv:
                assert kept == list(range(nb))
                continue
            assert kept[len(kept) - nbt:] == list(range(nbv, nb)) if nbt else True
            vid, vref = kept[:len(kept) - nbt], ref[:len(ref) - nbt]
            if static:
                # static part: what the union adds on top of the oracle's dynamic list; it must be in both
                dyn = set(sel["dyn_idx"][i, :sel["dyn_cnt"][i] - nbt].tolist())
                extra = set(vref) - dyn
                assert extra <= set(vid), f"row {i}: static blocks missing: {sorted(extra - set(vid))}"
                if set(vid) == set(vref):
                    rep.rows_checked += 1
                    continue
                if w.mode == "topp":
                    # The GPU's dynamic prefix may be shorter or longer than the oracle's where the running
                    # mass sits on p (fp32 against fp64), and blocks the oracle counts as dynamic may be
                    # static on the GPU side.  What is unique: the list holds a top prefix of the oracle's
                    # order that carries the mass, and nothing outside the oracle's united list except
                    # blocks at the cut.
                    S_i, P_i = sel["S"][i], sel["P"][i]
                    order = sorted(range(nbv), key=lambda j: (-S_i[j], j))
                    K = set(vid)
                    q = 0
                    while q < nbv and order[q] in K:
                        q += 1
                    run = np.cumsum(P_i[order])
                    assert q > 0 and run[q - 1] >= value * (1 - CUT_MARGIN), f"row {i}: top prefix of {q} holds {run[q - 1] if q else 0}"
                    cut = S_i[order[q - 1]]
                    pos = {j: r for r, j in enumerate(order)}
                    for j in K - set(vref):
                        assert _near_topp_cut(S_i, run, pos, j, cut, value, margin), \
                            f"row {i}: block {j} is neither static nor near the cut"
                    rep.near_cut_blocks += len(K ^ set(vref))
                    rep.rows_checked += 1
                    continue
                if len(vref) == nbv:                   # a full row has no cut to be near
                    raise AssertionError(f"row {i}: expected every block")
                vid = sorted(set(vid) - extra)
                vref = sorted(dyn - extra)
                if w.mode != "topp":
                    k = len(vref)                      # dynamic picks that are not static as well
            if w.mode == "topp":
                _check_row_topp(sel["S"][i], sel["P"][i], vid, vref, value, rep, margin)
            else:
                assert len(vid) == k, f"row {i}: {len(vid)} kept, k = {k}"
                _check_row_topk(sel["S"][i], vid, vref, k, rep, margin)
            rep.rows_checked += 1
        spars.append(so.sparsity(w.grid, w.n_text, blk, kv_idx[bh, :nb], kv_cnt[bh, :nb]))
    rep.sparsity = float(np.mean(spars))


def sample_blocks(g: Dict[str, int], n: Optional[int], rng) -> List[int]:
    nb = g["NB"]
    if n is None or n >= nb:
        return list(range(nb))
    must = {0, 1, nb - 1, nb - 2, g["NBv"] - 1, g["nbw"] - 1, g["nbw"] * g["nbh"] - 1}
    must = {b for b in must if 0 <= b < nb}
    extra = set(int(x) for x in rng.choice(nb, max(0, n - len(must)), replace=False))
    return sorted(must | extra)


def check_attention(w: Workload, plan: binding.Plan, qb, kb, vb, O: torch.Tensor, scheme, rep: Report,
                    blocks_per_head: Optional[int] = None, rng=None, heads: Optional[Sequence[int]] = None):
    """Stage 4: the GPU's own lists are fed to the oracle (Eq. 2), outputs compared on the sampled blocks."""
    t = plan.tables()
    kv_idx, kv_cnt = t["kv_idx"].cpu().numpy(), t["kv_cnt"].cpu().numpy()
    Oh = O.detach().float().cpu().numpy().reshape(w.batch * w.heads, w.n_tokens, w.d)
    num = den = 0.0
    for bh in (range(w.batch * w.heads) if heads is None else heads):
        blk = w.candidates[scheme[bh]]
        g = so.geometry(w.grid, w.n_text, blk)
        qbl = sample_blocks(g, blocks_per_head, rng)
        out, tok = so.attention_blocks(qb[bh], kb[bh], vb[bh], w.grid, w.n_text, blk, qbl,
                                       kv_idx[bh, :g["NB"]], kv_cnt[bh, :g["NB"]])
        m = tok >= 0
        got = Oh[bh][tok[m]]
        ref = out[m]
        assert np.isfinite(got).all(), "non-finite attention output"
        diff = got - ref
        rep.attn_max_abs = max(rep.attn_max_abs, float(np.abs(diff).max()))
        num += float((diff ** 2).sum())
        den += float((ref ** 2).sum())
        rep.attn_blocks += len(qbl)
    rep.attn_rel_fro = max(rep.attn_rel_fro, float(np.sqrt(num / max(den, 1e-300))))
    assert rep.attn_max_abs <= ATTN_MAX_ABS, f"max-abs {rep.attn_max_abs}"
    assert rep.attn_rel_fro <= ATTN_REL_FRO, f"relative Frobenius {rep.attn_rel_fro}"


def run_layer_parity(w: Workload, forced=None, rows_per_head=None, blocks_per_head=None, seed=0,
                     attn_heads=None, static=None, estimator="mean", check_scores=True) -> Report:
    """All four stages through the C ABI, each checked against the oracle."""
    rng = np.random.default_rng(seed)
    rep = Report()
    Q, K, V = make_qkv(w, "cuda")
    O = torch.full_like(Q, float("nan"))
    BH = w.batch * w.heads
    qb = bf16_bits(Q).reshape(BH, w.n_tokens, w.d)
    kb = bf16_bits(K).reshape(BH, w.n_tokens, w.d)
    vb = bf16_bits(V).reshape(BH, w.n_tokens, w.d)
    plan = make_plan(w, static=static, estimator=estimator)
    try:
        plan.spade_plan(Q, K, forced_scheme=forced)
        scheme = check_plan(w, plan, qb, kb, rep, forced)
        plan.spade_summarize(Q, K)
        check_summaries(w, plan, qb, kb, scheme)
        plan.spade_select()
        if estimator != "mean" and check_scores:
            check_minmax(w, plan, qb, kb, scheme, estimator)
        check_select(w, plan, qb, kb, scheme, rep, rows_per_head, rng, static, estimator)
        plan.spade_attn(Q, K, V, O)
        plan.spade_status()
        torch.cuda.synchronize()
        check_attention(w, plan, qb, kb, vb, O, scheme, rep, blocks_per_head, rng, attn_heads)
        assert bool(torch.isfinite(O).all()), "some output rows were never written"
    finally:
        plan.close()
    return rep
