"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, stage by stage."""
import numpy as np
import pytest
import torch

from paper_2608_03335_b200.workloads import WORKLOADS, Workload, small_variant

pytestmark = pytest.mark.gpu


def _run(w, **kw):
    kw = dict(kw)
    from tests.parity_util import run_layer_parity
    rep = run_layer_parity(w, **kw)
    print(f"[{w.name}] rows {rep.rows_checked} near-cut {rep.near_cut_blocks} scheme-ties {rep.scheme_ties} "
          f"attn blocks {rep.attn_blocks} max-abs {rep.attn_max_abs:.3e} rel-fro {rep.attn_rel_fro:.3e} "
          f"sparsity {rep.sparsity:.4f} score-err {rep.score_err_rel:.2e} (kernel alone {rep.score_err_kernel:.2e}) of the magnitude bound")
    return rep


def test_tiny_topk():
    rep = _run(WORKLOADS["tiny"])
    assert rep.rows_checked == 2 * 16


def test_tiny_topp():
    _run(WORKLOADS["tiny_topp"])


@pytest.mark.parametrize("heads", [64, 200])
def test_many_heads_on_a_tiny_grid(heads):
    """More heads than the estimator has score tiles per SM: 64 heads give 64 tiles for 148 CTAs (ranges of zero
    and one tile), 200 heads give ranges of one or two tiles that cross from one head into the next; the
    plan-stage tables, the head ordering and the attention work list run with hundreds of heads as well."""
    w = small_variant(WORKLOADS["wan14b"], heads=heads, grid=(4, 8, 16))
    _run(w, rows_per_head=4, blocks_per_head=2, seed=23)


def test_wan_small_ragged_grid_argmax_scheme():
    # 5x14x20: every candidate has partial edge blocks along some axis; odd block counts
    w = small_variant(WORKLOADS["wan1p3b"], heads=3, grid=(5, 14, 20))
    _run(w)


def test_hunyuan_small_text_tokens_topp():
    # 100 text tokens: a ragged text block under both block sizes; 4 candidates incl. the temporal one
    w = small_variant(WORKLOADS["hunyuan"], heads=4, grid=(16, 9, 12), n_text=100)
    _run(w)


def test_hunyuan_small_text_tokens_topk():
    w = small_variant(WORKLOADS["hunyuan_topk"], heads=4, grid=(16, 9, 12), n_text=100)
    _run(w)


def test_wan14b_small_three_head_classes():
    w = small_variant(WORKLOADS["wan14b"], heads=5, grid=(9, 10, 12))
    _run(w)


@pytest.mark.parametrize("cand", [0, 1, 2, 3])
@pytest.mark.parametrize("s", [0.0, 0.5, 0.95])
def test_forced_scheme_sparsity_sweep_small(cand, s):
    base = small_variant(WORKLOADS["wan14b"], heads=2, grid=(9, 10, 12))
    w = base.replace(name=f"sweep_small_c{cand}_s{s}", mode="sparsity", value=s)
    _run(w, forced=[cand] * 2)


def test_full_mask_equals_dense_attention():
    """Target sparsity 0 keeps every block: the output must equal plain softmax attention (Eq. 1)."""
    from paper_2608_03335_b200 import binding
    from paper_2608_03335_b200.workloads import make_qkv
    w = small_variant(WORKLOADS["wan14b"], heads=2, grid=(5, 9, 11)).replace(mode="sparsity", value=0.0)
    Q, K, V = make_qkv(w, "cuda")
    for cand in range(len(w.candidates)):
        O = torch.zeros_like(Q)
        plan = binding.Plan(w.batch, w.heads, w.grid, w.n_text, w.candidates, w.mode, w.value)
        plan.spade_forward(Q, K, V, O, forced_scheme=[cand] * w.heads)
        plan.spade_status()
        ref = torch.softmax(Q.double() @ K.double().transpose(-1, -2) / np.sqrt(w.d), -1) @ V.double()
        err = (O.double() - ref).abs().max().item()
        rel = ((O.double() - ref).norm() / ref.norm()).item()
        plan.close()
        assert err <= 2e-2 and rel <= 5e-3, (cand, err, rel)


@pytest.mark.parametrize("grid,cands", [((1, 8, 8), ((1, 8, 8),)),          # a single 64-token block
                                        ((1, 8, 16), ((1, 8, 16),)),        # a single 128-token block
                                        ((1, 3, 5), ((4, 4, 4),)),          # grid smaller than one block
                                        ((4, 4, 12), ((4, 4, 4),)),         # odd number of 64-token blocks
                                        ((2, 9, 17), ((2, 8, 8), (4, 4, 4)))])
def test_degenerate_grids(grid, cands):
    w = Workload("degenerate", 7, 2, grid, 0, cands, "topk", 2, "iso_2_6", 4.0)
    _run(w)


def test_batch_of_two_and_per_head_budgets():
    """B = 2 (heads of both batch items are independent units) and a different keep count per head."""
    from oracle import spade_oracle as so
    from paper_2608_03335_b200 import binding
    from paper_2608_03335_b200.workloads import bf16_bits, make_qkv
    w = small_variant(WORKLOADS["wan1p3b"], heads=2, grid=(4, 8, 20)).replace(batch=2, mode="topk", value=3)
    _run(w)
    per_head = [1.0, 2.0, 5.0, 7.0]
    Q, K, V = make_qkv(w, "cuda")
    O = torch.zeros_like(Q)
    plan = binding.Plan(w.batch, w.heads, w.grid, w.n_text, w.candidates, "topk", 3, per_head=per_head)
    plan.spade_forward(Q, K, V, O)
    plan.spade_status()
    t = plan.tables()
    scheme = t["scheme"].cpu().numpy()
    qb = bf16_bits(Q).reshape(4, w.n_tokens, w.d)
    kb = bf16_bits(K).reshape(4, w.n_tokens, w.d)
    for bh in range(4):
        blk = w.candidates[scheme[bh]]
        sel = so.select_head(qb[bh], kb[bh], w.grid, 0, blk, "topk", per_head[bh])
        nb = sel["geo"]["NB"]
        assert int(t["keep"][bh]) == min(int(per_head[bh]), nb)
        for i in range(nb):
            got = t["kv_idx"][bh, i, :int(t["kv_cnt"][bh, i])].cpu().tolist()
            assert got == sel["kv_idx"][i, :sel["kv_cnt"][i]].tolist()
    plan.close()


@pytest.mark.parametrize("static", [dict(window=1), dict(sink_tokens=70), dict(intra_threshold=0.35),
                                    dict(intra_threshold=0.35, window=0, sink_tokens=5)])
def test_static_and_intra_masks_united_with_the_selection(static):
    """Local window, attention sink and intra-block thresholding (Sec. 3.3) on top of Top-K / Top-P."""
    w = small_variant(WORKLOADS["wan14b"], heads=5, grid=(9, 10, 12))
    _run(w, static=static)
    _run(w.replace(mode="topp", value=0.6), static=static)
    _run(small_variant(WORKLOADS["hunyuan_topk"], heads=2, grid=(16, 9, 12), n_text=100), static=static, forced=[3, 1])


def test_eight_candidates():
    """The maximum number of blocking candidates, mixed 64- and 128-token blocks (their common cell is 1x1x4 tokens)."""
    cands = ((4, 4, 4), (2, 8, 8), (1, 8, 16), (8, 2, 4), (16, 1, 4), (1, 8, 8), (2, 4, 8), (4, 2, 16))
    w = Workload("eight", 9, 3, (8, 9, 18), 0, cands, "sparsity", 0.6, "aniso_bw_1_8", 6.0)
    _run(w)


def test_keep_one_and_keep_all():
    base = small_variant(WORKLOADS["wan1p3b"], heads=2, grid=(4, 8, 20))
    _run(base.replace(mode="topk", value=1))
    _run(base.replace(mode="topk", value=10_000))
    _run(base.replace(mode="topp", value=1.0))


@pytest.mark.parametrize("grid,mode,value", [((16, 32, 32), "sparsity", 0.8), ((16, 32, 32), "sparsity", 0.45), ((20, 32, 64), "sparsity", 0.8),
                                             ((16, 32, 32), "topp", 0.5), ((20, 32, 64), "topp", 0.9)])
def test_rows_with_ties_and_clusters_are_the_exact_top_of_the_table_lowest_ids_first(grid, mode, value):
    """Score rows that hold large groups of equal or nearly equal values (more than the 64 the index search ranks
    directly, so its histogram is refined between the group's own extremes, and rows where every score is the
    same): the list must agree with the oracle away from the cut, and be the exact top of the fp32 table the
    search read: nothing dropped scores higher than something kept, equal scores go by lower id.  Top-K keeps
    exactly k; Top-P keeps the shortest such prefix whose softmax mass reaches p (to 1e-4 of p: the search adds
    the masses in 2^-40 fixed point)."""
    from tests import parity_util as pu
    from oracle import spade_oracle as so
    from paper_2608_03335_b200.workloads import make_qkv, bf16_bits
    w = small_variant(WORKLOADS["wan14b"], heads=3, grid=grid).replace(mode=mode, value=value)
    blk = w.candidates[0]
    g = so.geometry(w.grid, w.n_text, blk)
    nbv = g["NBv"]
    assert nbv >= 256 and all(x % b == 0 for x, b in zip(grid, blk))
    Q, K, V = make_qkv(w, "cuda")
    K = K.clone()
    tok = [torch.as_tensor(so.block_tokens(w.grid, w.n_text, blk, b), device="cuda", dtype=torch.long) for b in range(nbv)]
    c0 = K[0, 0, tok[3][0]].clone()                    # head 0: blocks 0..99 made of one token value -> 100 equal scores per row
    for b in range(100):
        K[0, 0, tok[b]] = c0
    c1 = K[0, 1, tok[7][5]].clone()                    # head 1: every key the same -> every row one value
    K[0, 1, :, :] = c1
    c2 = K[0, 2, tok[11][1]].clone()                   # head 2: blocks 50..179 one value each, a bf16 step or two apart
    for b in range(50, 180):
        K[0, 2, tok[b]] = c2
        ch = (b * 5) % w.d
        step = c2[ch].abs().float() * 2.0 ** -7 + 2.0 ** -20
        K[0, 2, tok[b][: 1 + b // 64], ch] = (c2[ch].float() + step).to(torch.bfloat16)
    K = K.contiguous()
    BH = w.batch * w.heads
    qb, kb = (bf16_bits(x).reshape(BH, w.n_tokens, w.d) for x in (Q, K))
    plan = pu.make_plan(w)
    try:
        forced = [0, 0, 0]
        plan.spade_plan(Q, K, forced_scheme=forced)
        plan.spade_summarize(Q, K)
        plan.spade_select()
        plan.spade_status()
        torch.cuda.synchronize()
        rep = pu.Report()
        pu.check_select(w, plan, qb, kb, forced, rep)
        t = plan.tables()
        keep = t["keep"].cpu().numpy()
        kv_idx, kv_cnt = t["kv_idx"].cpu().numpy(), t["kv_cnt"].cpu().numpy()
        big_groups = 0
        for bh in range(BH):
            S = t["block_scores"][bh, :nbv, :nbv].cpu().numpy()
            for i in range(nbv):
                kept = kv_idx[bh, i, :kv_cnt[bh, i]].tolist()
                k = int(keep[bh]) if mode != "topp" else len(kept)
                order = sorted(range(nbv), key=lambda j: (-S[i, j], j))
                assert kept == sorted(order[:k]), f"head {bh} row {i}: not the top {k} by (score, lower id)"
                if mode == "topp":
                    wgt = np.exp(S[i, order].astype(np.float64) - float(S[i, order[0]]))
                    run = np.cumsum(wgt) / wgt.sum()
                    assert run[k - 1] >= value * (1 - 1e-4), f"head {bh} row {i}: kept mass {run[k - 1]} < p"
                    assert k == 1 or run[k - 2] <= value * (1 + 1e-4), f"head {bh} row {i}: a shorter prefix holds {run[k - 2]}"
                cut = S[i, order[k - 1]]
                big_groups += int((np.abs(S[i] - cut) <= 1e-3 * max(abs(cut), 1e-6)).sum() > 64)
        assert big_groups > nbv, "the inputs did not put large groups at the cut"
        print(f"[ties {grid} {mode} {value}] rows {rep.rows_checked} near-cut {rep.near_cut_blocks}, rows with > 64 values at the cut: {big_groups}")
    finally:
        plan.close()


@pytest.mark.parametrize("mode,value", [("sparsity", 0.9), ("topp", 0.8)])
def test_longest_rows_the_library_takes(mode, value):
    """2048 video blocks per head, the most a plan accepts: the index search holds 16 float4 per lane, the
    estimator walks 16 x 16 score tiles."""
    w = small_variant(WORKLOADS["wan14b"], heads=1, grid=(32, 64, 64)).replace(mode=mode, value=value)
    _run(w, forced=[0], rows_per_head=24, blocks_per_head=4, seed=17)


def test_caller_written_lists_and_empty_rows():
    """spade_attn on lists the caller wrote: random masks, and an empty row gives zeros."""
    from oracle import spade_oracle as so
    from paper_2608_03335_b200 import binding
    from paper_2608_03335_b200.workloads import bf16_bits, make_qkv
    w = small_variant(WORKLOADS["wan1p3b"], heads=2, grid=(4, 8, 20))
    rng = np.random.default_rng(5)
    Q, K, V = make_qkv(w, "cuda")
    for cand, blk in enumerate(w.candidates):
        g = so.geometry(w.grid, 0, blk)
        nb = g["NB"]
        plan = binding.Plan(w.batch, w.heads, w.grid, w.n_text, w.candidates, "topk", nb)
        plan.spade_plan(Q, K, forced_scheme=[cand] * w.heads)
        t = plan.tables()
        idx = np.full((w.heads, t["NBmax"], t["cap"]), -1, np.int32)
        cnt = np.zeros((w.heads, t["NBmax"]), np.int32)
        for h in range(w.heads):
            for i in range(nb):
                keep = np.nonzero(rng.random(nb) < 0.3)[0]
                if i == 1:
                    keep = keep[:0]                                    # empty row
                elif len(keep) == 0:
                    keep = np.array([i])
                cnt[h, i] = len(keep)
                idx[h, i, :len(keep)] = keep
        t["kv_idx"].copy_(torch.from_numpy(idx))
        t["kv_cnt"].copy_(torch.from_numpy(cnt))
        O = torch.full_like(Q, float("nan"))
        plan.spade_attn(Q, K, V, O)
        plan.spade_status()
        Oh = O.float().cpu().numpy().reshape(w.heads, w.n_tokens, w.d)
        for h in range(w.heads):
            blocks = [i for i in range(nb) if i != 1]
            out, tok = so.attention_blocks(bf16_bits(Q)[0, h], bf16_bits(K)[0, h], bf16_bits(V)[0, h], w.grid, 0, blk,
                                           blocks, idx[h, :nb], cnt[h, :nb])
            m = tok >= 0
            assert np.abs(Oh[h][tok[m]] - out[m]).max() <= 2e-2
            assert np.all(Oh[h][so.block_tokens(w.grid, 0, blk, 1)] == 0.0)
        plan.close()


# ---- full sizes, in the launch configuration bench.py times: sampled rows / blocks ------------------------
def test_full_size_wan1p3b_sampled():
    """The default bench workload: every head's scheme choice, AS and summaries in full; 24 list rows
    and 10 query blocks per head against the oracle."""
    rep = _run(WORKLOADS["wan1p3b"], rows_per_head=24, blocks_per_head=10, seed=11)
    assert abs(rep.sparsity - 0.80) < 0.02


def test_full_size_hunyuan_text_sampled():
    _run(WORKLOADS["hunyuan_topk"], rows_per_head=12, blocks_per_head=8, seed=12, attn_heads=[0, 5, 13, 23])


def test_full_size_hunyuan_topp_lists_sampled():
    _run(WORKLOADS["hunyuan"], rows_per_head=12, blocks_per_head=8, seed=14, attn_heads=[7])


def test_full_size_wan14b_sampled():
    _run(WORKLOADS["wan14b"], rows_per_head=8, blocks_per_head=8, seed=13, attn_heads=[0, 17, 39])


def test_full_size_paper_shapes_sampled():
    """The two shapes behind the paper's own latency numbers (up to 1804 blocks per head)."""
    _run(WORKLOADS["paper_wan"], rows_per_head=4, blocks_per_head=6, seed=15, attn_heads=[3])
    _run(WORKLOADS["paper_hunyuan"], rows_per_head=4, blocks_per_head=6, seed=16, attn_heads=[11])


@pytest.mark.parametrize("cand", [0, 1, 2, 3])
def test_full_size_sweep_forced_candidate_sparse(cand):
    """Config 5 at its full shape (40 heads, N = 75 600): every head forced onto one candidate, target
    sparsity 85 %.  Forced plans take the per-candidate summary pass instead of the cell tables; list
    rows and query blocks are sampled, attention on three heads."""
    from paper_2608_03335_b200.workloads import sweep_workload
    w = sweep_workload(cand, 0.85)
    rep = _run(w, forced=[cand] * w.heads, rows_per_head=6, blocks_per_head=8, seed=40 + cand, attn_heads=[0, 17, 39])
    assert abs(rep.sparsity - 0.85) < 0.03


@pytest.mark.parametrize("cand", [0, 1])
def test_full_size_sweep_full_mask_is_dense_attention(cand):
    """Config 5, target sparsity 0 on a 64-token and a 128-token candidate: every row lists every block
    (row capacity = block count, 1440 K units per work item for 4x4x4), so the oracle fed the GPU's lists
    evaluates Eq. 2 with M = 0, i.e. dense softmax attention (Eq. 1), on the sampled query blocks."""
    from paper_2608_03335_b200.workloads import sweep_workload
    w = sweep_workload(cand, 0.0)
    rep = _run(w, forced=[cand] * w.heads, rows_per_head=4, blocks_per_head=8, seed=50 + cand, attn_heads=[3, 38])
    assert abs(rep.sparsity) < 1e-12
    assert rep.near_cut_blocks == 0


def test_full_size_sweep_sparsest_point():
    """Config 5 at 95 %: the shortest lists (72 of 1440 blocks for 4x4x4)."""
    from paper_2608_03335_b200.workloads import sweep_workload
    w = sweep_workload(0, 0.95)
    _run(w, forced=[0] * w.heads, rows_per_head=6, blocks_per_head=8, seed=60, attn_heads=[11])


@pytest.mark.parametrize("estimator", ["dsa", "dsa2"])
def test_minmax_estimators_tiny_and_ragged(estimator):
    """Max / min summaries (bit-exact), the estimator's scores, the lists and the attention output."""
    _run(WORKLOADS["tiny"], estimator=estimator)
    _run(WORKLOADS["tiny_topp"], estimator=estimator)
    _run(small_variant(WORKLOADS["hunyuan_topk"], heads=3, grid=(16, 9, 12), n_text=100), estimator=estimator)


@pytest.mark.parametrize("estimator", ["dsa", "dsa2"])
def test_minmax_estimators_several_score_tiles(estimator):
    # 10x30x44 tokens: 200+ blocks per head under every candidate, so the 64 x 64 score tiles have a ragged tail
    w = small_variant(WORKLOADS["wan14b"], heads=3, grid=(10, 30, 44))
    _run(w, estimator=estimator, rows_per_head=24, blocks_per_head=6, seed=21)


def test_minmax_estimator_with_static_masks():
    w = small_variant(WORKLOADS["wan14b"], heads=2, grid=(9, 10, 12))
    _run(w, estimator="dsa", static=dict(window=1, sink_tokens=70))


def test_full_size_wan1p3b_minmax_estimator_sampled():
    _run(WORKLOADS["wan1p3b"], estimator="dsa", rows_per_head=12, blocks_per_head=4, seed=22, attn_heads=[0, 7])
    _run(WORKLOADS["wan1p3b"], estimator="dsa2", rows_per_head=12, blocks_per_head=4, seed=23, attn_heads=[5])


def test_estimator_argument_is_validated():
    from paper_2608_03335_b200 import binding
    w = WORKLOADS["tiny"]
    plan = binding.Plan(w.batch, w.heads, w.grid, w.n_text, w.candidates, w.mode, w.value)
    try:
        assert binding.lib().spade_plan_set_estimator(plan.handle, 7) == -1
        assert b"estimator" in binding.lib().spade_last_error()
        assert binding.lib().spade_plan_set_estimator(plan.handle, 2) == 0
    finally:
        plan.close()


def test_layer_can_be_captured_in_a_cuda_graph_and_replayed():
    """The four calls only enqueue work on the given stream, so a caller can capture one layer and replay it."""
    from paper_2608_03335_b200 import binding
    from paper_2608_03335_b200.workloads import make_qkv
    w = small_variant(WORKLOADS["wan1p3b"], heads=3, grid=(5, 14, 20))
    Q, K, V = make_qkv(w, "cuda")
    O = torch.empty_like(Q)
    plan = binding.Plan(w.batch, w.heads, w.grid, w.n_text, w.candidates, w.mode, w.value)
    try:
        def layer(stream=None):
            plan.spade_plan(Q, K, stream=stream)
            plan.spade_summarize(Q, K, stream=stream)
            plan.spade_select(stream=stream)
            plan.spade_attn(Q, K, V, O, stream=stream)
        layer()
        torch.cuda.synchronize()
        eager = O.clone()
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(s):
            with torch.cuda.graph(g, stream=s):
                layer(stream=s)
        for _ in range(2):
            O.fill_(float("nan"))
            g.replay()
            torch.cuda.synchronize()
            assert torch.equal(O, eager)
        plan.spade_status()
    finally:
        plan.close()


def test_captured_layer_with_forced_schemes_keeps_them_after_the_host_list_is_gone():
    """Forced schemes travel inside the launch: a captured layer replays the schemes it was captured with,
    whatever happens to the caller's (here pinned, then overwritten) host array afterwards."""
    import ctypes as C
    from paper_2608_03335_b200 import binding
    from paper_2608_03335_b200.workloads import make_qkv
    w = small_variant(WORKLOADS["wan14b"], heads=4, grid=(9, 10, 12))
    Q, K, V = make_qkv(w, "cuda")
    O = torch.empty_like(Q)
    forced = [3, 0, 2, 1]
    plan = binding.Plan(w.batch, w.heads, w.grid, w.n_text, w.candidates, w.mode, w.value)
    try:
        plan.spade_forward(Q, K, V, O, forced_scheme=forced)
        torch.cuda.synchronize()
        eager = O.clone()
        host = torch.tensor(forced, dtype=torch.int32).pin_memory()           # truly asynchronous if it were copied
        ptr = C.cast(host.data_ptr(), C.POINTER(C.c_int32))
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(s):
            with torch.cuda.graph(g, stream=s):
                binding._check(binding.lib().spade_forward(plan.handle, binding._ptr(Q), binding._ptr(K), binding._ptr(V),
                                                            binding._ptr(O), plan._ws_ptr, binding._stream(s), ptr))
        host.fill_(1)                                                          # the caller's list changes ...
        for _ in range(2):
            O.fill_(float("nan"))
            g.replay()
            torch.cuda.synchronize()
            assert plan.tables()["scheme"].cpu().tolist() == forced           # ... the replay does not
            assert torch.equal(O, eager)
        plan.spade_status()
    finally:
        plan.close()


@pytest.mark.parametrize("heads,pinned", [(5, True), (6, False), (9, True), (2, True), (13, True), (33, True)])
def test_host_entry_point_matches_the_device_path(heads, pinned):
    """spade_forward_host (head chunks, copies overlapped with kernels) gives the bytes spade_forward gives."""
    from paper_2608_03335_b200 import binding
    from paper_2608_03335_b200.workloads import make_qkv
    w = small_variant(WORKLOADS["hunyuan_topk"], heads=heads, grid=(16, 9, 12), n_text=100)
    Q, K, V = make_qkv(w, "cuda")
    O = torch.empty_like(Q)
    plan = binding.Plan(w.batch, w.heads, w.grid, w.n_text, w.candidates, w.mode, w.value)
    try:
        plan.spade_forward(Q, K, V, O)
        plan.spade_status()
        ref = O.clone()
        hq, hk, hv = (x.cpu() for x in (Q, K, V))
        ho = torch.zeros_like(hq)
        if pinned:
            hq, hk, hv, ho = (x.pin_memory() for x in (hq, hk, hv, ho))
        dQ, dK, dV, dO = (torch.zeros_like(Q) for _ in range(4))
        for _ in range(2):
            ho.fill_(float("nan"))
            plan.spade_forward_host(hq, hk, hv, ho, dQ, dK, dV, dO)
            assert torch.equal(ho, ref.cpu())
        plan.spade_status()
        # forced schemes are split per chunk as well
        forced = [i % len(w.candidates) for i in range(heads)]
        plan.spade_forward(Q, K, V, O, forced_scheme=forced)
        ref = O.clone()
        plan.spade_forward_host(hq, hk, hv, ho, dQ, dK, dV, dO, forced_scheme=forced)
        assert torch.equal(ho, ref.cpu())
        # the device path still works on this plan afterwards
        plan.spade_forward(Q, K, V, O, forced_scheme=forced)
        torch.cuda.synchronize()
        assert torch.equal(O, ref)
    finally:
        plan.close()


def test_topp_one_keeps_the_mass_without_overrunning_the_histograms():
    """p = 1: the crossing of the cumulative mass is decided by rounding; the histogram search must still
    land on a non-empty bin in every pass (regression: an empty bin left the next pass without keys)."""
    w = small_variant(WORKLOADS["wan14b"], heads=4, grid=(15, 18, 25)).replace(mode="topp", value=1.0)
    _run(w, forced=[0, 3, 2, 3], rows_per_head=40, blocks_per_head=4, seed=31)
    _run(WORKLOADS["tiny_topp"].replace(value=1.0))
    _run(small_variant(WORKLOADS["hunyuan"], heads=3, grid=(16, 9, 12), n_text=100).replace(value=0.999))


def test_running_maximum_that_keeps_growing_rescales_output_and_row_sums():
    """K grows along the sequence, so every few units the running maximum of a row jumps by more than the
    lazy-rescale threshold: O and the row sums kept by the tensor core are rescaled many times per tile."""
    from tests import parity_util as pu
    from paper_2608_03335_b200.workloads import make_qkv, bf16_bits
    for base, grid in (("wan14b", (6, 12, 16)), ("wan1p3b", (4, 16, 16))):
        w = small_variant(WORKLOADS[base], heads=2, grid=grid).replace(mode="sparsity", value=0.3)
        Q, K, V = make_qkv(w, "cuda")
        ramp = torch.linspace(1.0, 24.0, w.n_tokens, device="cuda").view(1, 1, -1, 1)
        K = (K.float() * ramp).to(torch.bfloat16).contiguous()
        O = torch.full_like(Q, float("nan"))
        BH = w.batch * w.heads
        qb, kb, vb = (bf16_bits(x).reshape(BH, w.n_tokens, w.d) for x in (Q, K, V))
        plan = pu.make_plan(w)
        try:
            forced = [0, 1] if base == "wan14b" else [0, 2]          # a 64-token and a 128-token scheme
            plan.spade_plan(Q, K, forced_scheme=forced)
            plan.spade_summarize(Q, K)
            plan.spade_select()
            plan.spade_attn(Q, K, V, O)
            plan.spade_status()
            torch.cuda.synchronize()
            rep = pu.Report()
            pu.check_attention(w, plan, qb, kb, vb, O, forced, rep, None, np.random.default_rng(5))
            assert bool(torch.isfinite(O).all())
            print(f"[ramp {base}] attn blocks {rep.attn_blocks} max-abs {rep.attn_max_abs:.3e} rel-fro {rep.attn_rel_fro:.3e}")
        finally:
            plan.close()


def test_bounded_wait_gives_up_and_the_context_survives():
    """Failure detection without a fault: a wait on a barrier nothing completes returns after its limit."""
    import time
    from paper_2608_03335_b200 import binding
    t0 = time.perf_counter()
    r = binding.spade_selftest_bounded_wait(limit_us=2000)
    dt = time.perf_counter() - t0
    assert r["gave_up"] == 1 and r["abort_flag"] == 1
    assert 1_000_000 < r["cycles"] < 40_000_000            # ~2 ms at 1-2 GHz (the bound is limit * 2 cycles/ns)
    assert dt < 5.0
    x = torch.ones(8, device="cuda")                        # the context still works
    assert float(x.sum()) == 8.0


def test_policy_budget_follows_the_aggregation_score():
    """SPADE_POLICY_AS: per-head keep counts computed on the device from the selected scores."""
    from oracle import spade_oracle as so
    from paper_2608_03335_b200 import binding
    from paper_2608_03335_b200.workloads import bf16_bits, make_qkv
    from tests import parity_util as pu
    w = small_variant(WORKLOADS["wan14b"], heads=6, grid=(9, 10, 12))
    Q, K, V = make_qkv(w, "cuda")
    O = torch.full_like(Q, float("nan"))
    qb, kb, vb = (bf16_bits(x).reshape(w.heads, w.n_tokens, w.d) for x in (Q, K, V))
    plan = binding.Plan(w.batch, w.heads, w.grid, w.n_text, w.candidates, "policy_as", 0.7, gain=2.0)
    try:
        plan.spade_forward(Q, K, V, O)
        plan.spade_status()
        t = plan.tables()
        scheme = t["scheme"].cpu().numpy()
        keep = t["keep"].cpu().numpy()
        plans = [so.plan_head(qb[h], kb[h], w.grid, 0, w.candidates) for h in range(w.heads)]
        assert [p["scheme"] for p in plans] == scheme.tolist()
        sel_scores = [p["score"][p["scheme"]] for p in plans]
        nkb = [so.geometry(w.grid, 0, w.candidates[c])["NBv"] for c in scheme]
        k_ref, f = so.policy_keep_counts(sel_scores, nkb, float(np.float32(0.7)), 2.0)
        assert len(set(keep.tolist())) > 1                               # the policy does differentiate heads
        for h in range(w.heads):
            if keep[h] != k_ref[h]:                                      # fp32 scores may move a value sitting on an integer
                assert abs(keep[h] - k_ref[h]) == 1 and abs(f[h] * nkb[h] - round(f[h] * nkb[h])) < 1e-3
        rep = pu.Report()
        for h in range(w.heads):
            blk = w.candidates[scheme[h]]
            sel = so.select_head(qb[h], kb[h], w.grid, 0, blk, "topk", int(keep[h]))
            for i in range(nkb[h]):
                got = t["kv_idx"][h, i, :int(t["kv_cnt"][h, i])].cpu().tolist()
                pu._check_row_topk(sel["S"][i], got, sel["kv_idx"][i, :sel["kv_cnt"][i]].tolist(), int(keep[h]), rep)
        pu.check_attention(w, plan, qb, kb, vb, O, scheme, rep)
    finally:
        plan.close()


def test_topp_lists_are_reproducible_bit_for_bit_also_through_a_graph():
    """The Top-P index search adds the softmax mass of a histogram bin in fixed point, so the lists do not depend on
    the order in which lanes reach a bin: two eager runs and two replays of a captured layer give identical
    kv_idx / kv_cnt (and outputs)."""
    from paper_2608_03335_b200 import binding
    from paper_2608_03335_b200.workloads import make_qkv
    w = small_variant(WORKLOADS["hunyuan"], heads=4, grid=(16, 18, 24), n_text=100)
    Q, K, V = make_qkv(w, "cuda")
    O = torch.empty_like(Q)
    plan = binding.Plan(w.batch, w.heads, w.grid, w.n_text, w.candidates, w.mode, w.value)
    try:
        def layer(stream=None):
            plan.spade_plan(Q, K, stream=stream)
            plan.spade_summarize(Q, K, stream=stream)
            plan.spade_select(stream=stream)
            plan.spade_attn(Q, K, V, O, stream=stream)
        runs = []
        for _ in range(2):
            layer()
            torch.cuda.synchronize()
            t = plan.tables()
            runs.append((t["kv_idx"].clone(), t["kv_cnt"].clone(), O.clone()))
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(s):
            with torch.cuda.graph(g, stream=s):
                layer(stream=s)
        for _ in range(2):
            O.fill_(float("nan"))
            g.replay()
            torch.cuda.synchronize()
            t = plan.tables()
            runs.append((t["kv_idx"].clone(), t["kv_cnt"].clone(), O.clone()))
        cnt0 = runs[0][1]
        valid = torch.arange(runs[0][0].shape[2], device="cuda")[None, None, :] < cnt0[:, :, None]
        for idx, cnt, out in runs[1:]:
            assert torch.equal(cnt, cnt0)
            assert torch.equal(idx[valid], runs[0][0][valid])
            assert torch.equal(out, runs[0][2])
        plan.spade_status()
    finally:
        plan.close()


@pytest.mark.gpu
@pytest.mark.parametrize("grid,cand", [((21, 45, 80), (8, 2, 4)), ((21, 45, 80), (4, 4, 4)), ((16, 45, 80), (16, 1, 4)),
                                       ((5, 7, 9), (1, 1, 64)), ((1, 8, 8), (1, 8, 8)), ((3, 3, 3), (4, 4, 4))])
def test_tile_table_of_a_64_token_scheme_covers_every_block_once_whatever_the_cells_choose(grid, cand):
    from paper_2608_03335_b200 import binding
    # the attention stage pairs 64-token query blocks inside 2 x 2 x 2 cells of the block grid, along an axis chosen per
    # cell: for every axis the tiles of a cell must hold each of its blocks exactly once, partners one step along that
    # axis, and the tile count may not depend on the choice
    plan = binding.Plan(1, 1, grid, 0, (cand,), "sparsity", 0.5)
    g = plan.geometry(0)
    nbt, nbh, nbw = g["nbt"], g["nbh"], g["nbw"]
    tile_cell, pairs = plan.pair_table(0)
    assert tile_cell.shape[0] == pairs.shape[0]
    assert (tile_cell[1:] >= tile_cell[:-1]).all(), "the tiles of a cell are consecutive"
    nct, nch, ncw = (nbt + 1) // 2, (nbh + 1) // 2, (nbw + 1) // 2
    assert int(tile_cell.max()) + 1 == nct * nch * ncw
    stride = (nbh * nbw, nbw, 1)
    for a in range(3):
        seen = torch.zeros(g["NBv"], dtype=torch.int64)
        for t in range(pairs.shape[0]):
            e = int(pairs[t, a])
            qb0, qb1 = e & 0xffff, e >> 16
            cell = int(tile_cell[t])
            blocks = [qb0] if qb1 == 0xffff else [qb0, qb1]
            if qb1 != 0xffff:
                assert qb1 - qb0 in stride, "partners are neighbours along one axis"
            for b in blocks:
                it, ih, iw = b // (nbh * nbw), (b // nbw) % nbh, b % nbw
                assert ((it // 2) * nch + ih // 2) * ncw + iw // 2 == cell, "both blocks lie in the tile's cell"
                seen[b] += 1
        assert (seen == 1).all(), f"axis {a}: every video block in exactly one tile"
