"""Basis files (the offline "one-time SVD" result, Eq. 7) and state check-pointing: the state is a
flat caller-owned buffer, so a copy of its bytes taken between two steps resumes the run exactly."""
import numpy as np
import pytest
import torch

from paper_2601_07396_b200 import basis_io


def test_basis_file_round_trip(tmp_path):
    g = torch.Generator().manual_seed(0)
    V = torch.linalg.qr(torch.randn(96, 16, generator=g, dtype=torch.float64))[0].float()
    lam = torch.linspace(9.0, 1.0, 16, dtype=torch.float64)
    path = str(tmp_path / "block0.svcb")
    basis_io.save_basis(path, V, lam, 123.5)
    V2, lam2, tr = basis_io.load_basis(path)
    assert torch.equal(V, V2) and torch.equal(lam, lam2) and tr == 123.5
    assert (tmp_path / "block0.svcb").stat().st_size == 8 + 16 + 8 * 16 + 4 * 96 * 16
    with open(path, "r+b") as fh:      # a truncated or foreign file is refused
        fh.truncate(100)
    with pytest.raises(ValueError):
        basis_io.load_basis(path)
    (tmp_path / "junk").write_bytes(b"not a basis file at all")
    with pytest.raises(ValueError):
        basis_io.load_basis(str(tmp_path / "junk"))
    with pytest.raises(ValueError):
        basis_io.save_basis(path, V, lam[:5], 1.0)


@pytest.mark.gpu
def test_state_copy_resumes_the_trajectory_bit_for_bit(tmp_path):
    from paper_2601_07396_b200 import binding as sc
    from paper_2601_07396_b200 import streams
    spec = streams.StreamSpec("ckpt", blocks=1, rows=700, D=1024, dtype="bf16", k=64, T=8, interval=2, rank=128,
                              amp=30.0, power=1.0, noise_std=0.02)
    st = streams.BlockStream(spec, 0, device="cuda")
    N, D, k, dt = 700, 1024, 64, sc.BF16
    stack = streams.BlockStream(spec, 0, trajectory=1, device="cuda").features(0)
    Vk, lam, tr, _ = sc.svdcache_calibrate(stack, k)
    path = str(tmp_path / "b.svcb")
    basis_io.save_basis(path, Vk, lam, float(tr.cpu()[0]))
    Vl, laml, trl = basis_io.load_basis(path, device="cuda")
    assert torch.equal(Vl, Vk) and torch.equal(laml, lam)
    basis = sc.svdcache_basis_prepare(Vl, dt)
    for x, y in zip(sc.basis_views(basis, D, k, dt), sc.basis_views(sc.svdcache_basis_prepare(Vk, dt), D, k, dt)):
        assert torch.equal(x, y)     # (the padding between the sections is never written)

    def run(state, ts, out):
        for t in ts:
            if t % 2 == 0:
                sc.svdcache_full_step(st.features(t), basis, state, k, 0.9)
            else:
                sc.svdcache_cached_step(state, basis, out, k)

    ref_state = sc.new_state(N, D, k, dt, "cuda")
    ref_out = torch.empty(N, D, dtype=torch.bfloat16, device="cuda")
    run(ref_state, range(8), ref_out)
    a = sc.new_state(N, D, k, dt, "cuda")
    out = torch.empty_like(ref_out)
    run(a, range(0, 5), out)
    saved = a.cpu().clone()                 # the checkpoint: the state's bytes
    b = saved.to("cuda")                    # ... restored into another buffer
    run(b, range(5, 8), out)
    torch.cuda.synchronize()
    assert torch.equal(out, ref_out)
    for x, y in zip(sc.state_views(b, N, D, k, dt), sc.state_views(ref_state, N, D, k, dt)):
        assert torch.equal(x, y)
    assert sc.svdcache_state_query(b) == sc.svdcache_state_query(ref_state) == (4, 0)
