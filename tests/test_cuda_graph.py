"""The step calls only enqueue work on the caller's stream (no allocation, no synchronisation), so a
whole caching interval can be captured into a CUDA graph once and replayed: the launch-bound small
configurations (DiT-XL: 28 blocks of 2048 rows) pay one graph launch per interval instead of one
launch per kernel."""
import pytest
import torch

from paper_2601_07396_b200 import binding as sc
from paper_2601_07396_b200 import streams

pytestmark = pytest.mark.gpu


def test_an_interval_captured_in_a_cuda_graph_replays_the_eager_results():
    spec = streams.DIT_XL
    nb, N, D, k, dt = 4, spec.rows, spec.D, spec.k, sc.BF16
    strs = [streams.BlockStream(spec, b, device="cuda") for b in range(nb)]
    bases = torch.stack([sc.svdcache_basis_prepare(s.V_gen[:, :k].float().contiguous(), dt) for s in strs])
    F = torch.empty(nb, N, D, dtype=torch.bfloat16, device="cuda")
    outs = [torch.empty_like(F) for _ in range(2)]

    def interval(state, out_list):
        sc.svdcache_full_step_batched(F, bases, state, k, spec.beta)
        for o in out_list:
            sc.svdcache_cached_step_batched(state, bases, o, k)

    # eager reference over three intervals
    st_e = sc.new_state(N, D, k, dt, "cuda", blocks=nb)
    eager = []
    for t in (0, 4, 8):
        for b in range(nb):
            strs[b].features(t, out=F[b])
        interval(st_e, outs)
        eager.append(outs[1].clone())
    # the same three intervals as replays of one captured graph
    st_g = sc.new_state(N, D, k, dt, "cuda", blocks=nb)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):          # warm-up outside the capture (first-call set-up of the library)
        for b in range(nb):
            strs[b].features(0, out=F[b])
        interval(sc.new_state(N, D, k, dt, "cuda", blocks=nb), outs)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    launches0 = sc.svdcache_kernel_launches()
    with torch.cuda.graph(graph):
        interval(st_g, outs)
    assert sc.svdcache_kernel_launches() - launches0 == 3      # recorded, not run
    for i, t in enumerate((0, 4, 8)):
        for b in range(nb):
            strs[b].features(t, out=F[b])
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(outs[1], eager[i])
    for b in range(nb):
        assert sc.svdcache_state_query(st_g[b]) == (3, 0)
        for x, y in zip(sc.state_views(st_g[b], N, D, k, dt), sc.state_views(st_e[b], N, D, k, dt)):
            assert torch.equal(x, y)
