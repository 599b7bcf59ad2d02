"""The synthetic stream generators: determinism, shapes, and the structure they promise."""
import numpy as np
import torch

from paper_2601_07396_b200 import streams


def _small():
    return streams.StreamSpec("probe", blocks=2, rows=96, D=64, dtype="bf16", k=8, T=6,
                              interval=3, rank=16, amp=20.0, power=1.0, noise_std=0.02,
                              frame_rows=40, calib_trajectories=(1, 2), calib_timesteps=(0, 3))


def test_specs_match_the_five_configurations():
    s = streams.SPECS
    assert (s["tiny"].rows, s["tiny"].D, s["tiny"].k, s["tiny"].dtype) == (256, 1152, 32, "f32")
    assert s["tiny"].full_timesteps() == [0, 3, 6, 9]
    assert (s["dit_xl"].blocks, s["dit_xl"].rows, s["dit_xl"].k, s["dit_xl"].interval) == (28, 2048, 64, 4)
    assert (s["flux"].blocks, s["flux"].rows, s["flux"].D, s["flux"].k) == (57, 4608, 3072, 64)
    assert s["flux"].calib_rows() == 64 * 4608
    assert (s["hunyuan"].blocks, s["hunyuan"].rows, s["hunyuan"].k) == (60, 33 * 45 * 80, 128)
    assert len(s["flux"].full_timesteps()) == 9
    assert all(sp.beta == 0.9 for sp in s.values())


def test_stream_is_deterministic_and_typed():
    spec = _small()
    a = streams.BlockStream(spec, 1).features(2)
    b = streams.BlockStream(spec, 1).features(2)
    assert a.dtype == torch.bfloat16 and a.shape == (96, 64)
    assert torch.equal(a, b)
    c = streams.BlockStream(spec, 0).features(2)
    assert not torch.equal(a, c)


def test_basis_is_shared_across_trajectories_and_noise_flips_sign():
    spec = _small()
    s0 = streams.BlockStream(spec, 1, trajectory=0)
    s1 = streams.BlockStream(spec, 1, trajectory=1)
    assert torch.equal(s0.V_gen, s1.V_gen) and torch.equal(s0.s, s1.s)
    assert not torch.equal(s0.omega, s1.omega)
    V = s0.V_gen.numpy()
    np.testing.assert_allclose(V.T @ V, np.eye(spec.rank), atol=1e-12)
    # the part of F outside the generator basis is the noise, with alternating sign
    P = np.eye(spec.D) - V @ V.T
    f32 = streams.StreamSpec(**{**spec.__dict__, "dtype": "f32"})
    st = streams.BlockStream(f32, 1)
    e0 = st.features(0).double().numpy() @ P
    e1 = st.features(1).double().numpy() @ P
    np.testing.assert_allclose(e0, -e1, atol=1e-4)
    assert abs(e0.std() - spec.noise_std) < 0.3 * spec.noise_std


def test_calibration_stack_and_row_samples():
    spec = _small()
    stack = streams.calibration_stack(spec, 0)
    assert stack.shape == (2 * 2 * 96, 64) and stack.dtype == torch.bfloat16
    first = streams.BlockStream(spec, 0, trajectory=1).features(0)
    assert torch.equal(stack[:96], first)
    rows = streams.sample_rows(1000, 64, tile=128, extra=(500,))
    assert len(rows) == 64 and len(set(rows.tolist())) == 64
    for r in (0, 999, 127, 128, 895, 896, 500):
        assert r in rows.tolist()
    assert streams.sample_rows(10, 64).tolist() == list(range(10))
