"""The allocation-free Aggregation-Score entry point against the CPU oracle and the planning stage.

Collected last on purpose (file name): if it fails, a run that stops at the first failure has
already run everything else.  The entry point is for callers that cannot obtain device memory when
they need the scores -- code hosted inside a framework whose allocator owns the device, services on
a fixed memory budget -- so the test also checks, with the driver's own count of free device memory,
that repeated calls take none.
"""
import numpy as np
import pytest
import torch

from paper_2608_03335_b200.workloads import WORKLOADS, bf16_bits, make_qkv, small_variant

pytestmark = pytest.mark.gpu

RTOL = 2e-5       # the suite's tolerance for fp32 sums of bf16 rows against fp64


def _oracle_as(w, Q, K):
    """AS(Q|c), AS(K|c) of every head and candidate by the oracle (Eq. 3 over Eq. 4 / Algorithm 1)."""
    from oracle import spade_oracle as so
    BH = w.batch * w.heads
    qb = bf16_bits(Q).reshape(BH, w.n_tokens, w.d)
    kb = bf16_bits(K).reshape(BH, w.n_tokens, w.d)
    ref = np.zeros((BH, len(w.candidates), 2))
    for bh in range(BH):
        for c, blk in enumerate(w.candidates):
            ref[bh, c, 0] = so.aggregation_score(qb[bh], w.grid, w.n_text, blk)
            ref[bh, c, 1] = so.aggregation_score(kb[bh], w.grid, w.n_text, blk)
    return ref


@pytest.mark.parametrize("name,heads,grid,n_text", [("wan14b", 5, (9, 10, 12), 0), ("hunyuan_topk", 3, (16, 9, 12), 100)])
def test_noalloc_scores_match_the_oracle_and_the_planning_stage_twice_in_a_row(name, heads, grid, n_text):
    from paper_2608_03335_b200 import binding
    w = small_variant(WORKLOADS[name], heads=heads, grid=grid, n_text=n_text)
    Q, K, _ = make_qkv(w, "cuda")
    ref = _oracle_as(w, Q, K)
    plan = binding.Plan(w.batch, w.heads, w.grid, w.n_text, w.candidates, w.mode, w.value)
    try:
        plan.spade_plan(Q, K)                                   # the existing entry point
        torch.cuda.synchronize()
        planned = plan.tables()["as_"].clone()
        np.testing.assert_allclose(planned.cpu().numpy(), ref, rtol=RTOL)
        out = torch.empty_like(planned)
        side = torch.cuda.Stream()                              # a stream of the caller's, not the current one
        free_before = None
        for call in range(3):                                   # calls in a row share the built-in scratch
            if call == 1:
                # The first round has looked the scratch up and let torch's caching allocator take what the
                # checks below need; from here on the driver's count of free memory must not move.
                free_before = torch.cuda.mem_get_info()[0]
            out.fill_(float("nan"))
            torch.cuda.synchronize()
            plan.spade_aggregation_scores_noalloc(Q, K, out, stream=side if call == 2 else None)
            torch.cuda.synchronize()
            assert torch.isfinite(out).all()
            np.testing.assert_allclose(out.cpu().numpy(), ref, rtol=RTOL)                  # Eq. 3, against the oracle
            # the planning stage adds the same block values in another order (cells first): fp32 rounding apart
            torch.testing.assert_close(out, planned, rtol=RTOL, atol=1e-4)
        assert torch.cuda.mem_get_info()[0] == free_before
        # a second, different input must not see stale values of the first
        Q2, K2 = K.clone(), Q.clone()
        plan.spade_aggregation_scores_noalloc(Q2, K2, out)
        torch.cuda.synchronize()
        np.testing.assert_allclose(out.cpu().numpy(), ref[:, :, ::-1], rtol=RTOL)
        assert not np.allclose(ref, ref[:, :, ::-1])
    finally:
        plan.close()


def test_noalloc_rejects_plans_beyond_the_built_in_scratch():
    from paper_2608_03335_b200 import binding
    big = WORKLOADS["wan14b"].replace(heads=120)                # 120 x 4 x 2 x 1440 = 1 382 400 floats > 1 048 576
    plan = binding.Plan(big.batch, big.heads, big.grid, big.n_text, big.candidates, big.mode, big.value)
    try:
        x = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
        out = torch.zeros(big.heads, len(big.candidates), 2, device="cuda")
        with pytest.raises(binding.SpadeError) as e:
            plan.spade_aggregation_scores_noalloc(x, x, out)
        assert e.value.code == -2 and "scratch" in str(e.value)
    finally:
        plan.close()
