"""Row-sharded calibration: the host logic as two gloo ranks on the CPU (row ranges, the sum of
the partial Gram matrices by one all-reduce), and, on a GPU, the one-rank path against the plain
calibration and the cross-"prompt" similarity statistic of Fig. 1(b) against the oracle."""
import json
import os
import sys
import textwrap

import numpy as np
import pytest
import torch

from oracle import svdcache_oracle as oracle
from paper_2601_07396_b200 import sharded
from tests.test_bench_multirank import ROOT, _launch

WORKER = textwrap.dedent("""
    import json, sys
    sys.path.insert(0, %r)
    import numpy as np, torch, torch.distributed as dist
    from oracle import svdcache_oracle as oracle
    from paper_2601_07396_b200 import sharded
    import bench
    rank, world, _ = bench.dist_env()
    dist.init_process_group("gloo", rank=rank, world_size=world)
    rng = np.random.default_rng(7)                 # every rank draws the same stack
    M, D = 1001, 48
    F = rng.standard_normal((M, D))
    lo, hi = sharded.shard_rows(M, rank, world)
    G = torch.from_numpy(oracle.gram(F[lo:hi]))    # this rank's partial sum (Eq. 4 over its rows)
    sharded.allreduce_gram(G)
    total = oracle.gram(F)
    err = float(np.abs(G.numpy() - total).max() / np.abs(total).max())
    print(json.dumps({"rank": rank, "lo": lo, "hi": hi, "err": err, "trace": float(np.trace(G.numpy()))}))
    dist.destroy_process_group()
""") % ROOT


def test_row_ranges_are_disjoint_and_cover():
    for M, world in ((10, 3), (7, 8), (294912, 8), (0, 2), (5, 1)):
        parts = [sharded.shard_rows(M, r, world) for r in range(world)]
        assert parts[0][0] == 0 and parts[-1][1] == M
        assert all(a[1] == b[0] for a, b in zip(parts, parts[1:]))
        sizes = [hi - lo for lo, hi in parts]
        assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharded.shard_rows(10, 2, 2)


def test_two_ranks_sum_their_partial_gram_matrices():
    outs = _launch(WORKER, 2)
    rows = sorted((json.loads(o.strip().splitlines()[-1]) for o in outs), key=lambda r: r["rank"])
    assert (rows[0]["lo"], rows[0]["hi"], rows[1]["lo"], rows[1]["hi"]) == (0, 501, 501, 1001)
    assert rows[0]["err"] < 1e-14 and rows[1]["err"] < 1e-14
    assert rows[0]["trace"] == rows[1]["trace"]     # both ranks hold the same total


def test_similarity_statistic_of_the_oracle():
    """Fig. 1(b)'s measure on cases with known answers: identical decompositions give 1; a sign flip of
    a singular vector changes nothing; scaling the spectrum by c gives min(c, 1/c) for the singular
    values; orthogonal vectors give 0."""
    rng = np.random.default_rng(0)
    Q, _ = np.linalg.qr(rng.standard_normal((20, 6)))
    lam = np.array([9.0, 4.0, 1.0])
    V = Q[:, :3]
    assert oracle.basis_similarity(V, lam, V, lam)[:2] == pytest.approx((1.0, 1.0), abs=1e-14)
    assert oracle.basis_similarity(V, lam, -V, lam)[1] == pytest.approx(1.0, abs=1e-14)
    assert oracle.basis_similarity(V, lam, V, 4 * lam)[0] == pytest.approx(0.5, abs=1e-14)   # sigma doubled
    s, m, cols = oracle.basis_similarity(V, lam, Q[:, 3:], lam)
    assert m == pytest.approx(0.0, abs=1e-14) and np.allclose(cols, 0.0, atol=1e-14)
    # by hand: sigma_A = (3, 4), sigma_B = (4, 3): cos = 24/25, norms equal
    assert oracle.basis_similarity(V[:, :2], [9, 16], V[:, :2], [16, 9])[0] == pytest.approx(0.96, abs=1e-14)


@pytest.mark.gpu
def test_one_rank_sharded_calibration_is_the_plain_calibration():
    from paper_2601_07396_b200 import binding as sc
    from paper_2601_07396_b200 import streams
    spec = streams.StreamSpec("sh", blocks=1, rows=3000, D=384, dtype="bf16", k=32, T=2, interval=1,
                              rank=96, amp=40.0, power=1.1, noise_std=0.02)
    stack = streams.BlockStream(spec, 0, device="cuda").features(0)
    V0, l0, t0, _ = sc.svdcache_calibrate(stack, 32)
    V1, l1, t1, _ = sharded.calibrate_sharded(stack, 32)
    assert torch.equal(V0, V1) and torch.equal(l0, l1) and torch.equal(t0, t1)
    # two "ranks" by hand on one device: partial sums into two workspaces, added, finished
    D, k = 384, 32
    ws = [torch.empty(sc.svdcache_calibrate_workspace_bytes(D, k), dtype=torch.uint8, device="cuda") for _ in range(2)]
    for r in range(2):
        lo, hi = sharded.shard_rows(3000, r, 2)
        sc.svdcache_calibrate_begin(D, k, ws[r])
        sc.svdcache_calibrate_accumulate(stack[lo:hi], ws[r])
    sharded.gram_view(ws[0], D).add_(sharded.gram_view(ws[1], D))
    V2, l2, t2, _ = sc.svdcache_calibrate_finish(D, k, ws[0])
    Vo, lo_, to = oracle.calibrate(stack.double().cpu().numpy(), k)
    cos = np.linalg.svd(Vo.T @ V2.double().cpu().numpy(), compute_uv=False)
    assert cos.min() >= 1 - 1e-4
    np.testing.assert_allclose(l2.cpu().numpy(), lo_, rtol=1e-9)
    assert float(t2.cpu()[0]) == pytest.approx(to, rel=1e-12)


@pytest.mark.gpu
def test_decomposition_is_stable_across_synthetic_prompts():
    """Two calibration trajectories ("prompts") of one block share the generator's basis and spectrum:
    the statistic of Fig. 1(b), computed by the library, against the oracle's, and above the paper's
    0.8 mark for the singular values and for the leading, well separated singular vectors."""
    from paper_2601_07396_b200 import binding as sc
    from paper_2601_07396_b200 import streams
    spec = streams.DIT_XL
    k = 16
    res = []
    for traj in (1, 2):
        stack = streams.calibration_stack(spec, 3, device="cuda", trajectories=(traj,), rows_per_snapshot=1024)
        res.append(sc.svdcache_calibrate(stack, k)[:2])
    s_sig, s_vec, cols = sc.svdcache_basis_similarity(res[0][0], res[0][1], res[1][0], res[1][1])
    o_sig, o_vec, o_cols = oracle.basis_similarity(res[0][0].double().cpu().numpy(), res[0][1].cpu().numpy(),
                                                   res[1][0].double().cpu().numpy(), res[1][1].cpu().numpy())
    assert s_sig == pytest.approx(o_sig, abs=1e-12) and s_vec == pytest.approx(o_vec, abs=1e-9)
    np.testing.assert_allclose(cols.cpu().numpy(), o_cols, atol=1e-9)
    assert s_sig > 0.8 and cols[:4].min() > 0.8
