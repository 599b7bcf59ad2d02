"""The bounded waits of the tensor-core kernels: a wait that nothing will ever satisfy has
to give up by itself, leave SVDCACHE_ERR_TIMEOUT and the place of the wait in the state
header, and leave the device usable.  Nothing here faults or hangs: the kernel under test
waits about a millisecond on an mbarrier of its own and returns."""
import numpy as np
import pytest
import torch

from paper_2601_07396_b200 import binding as sc
from paper_2601_07396_b200 import streams
from tests.parity_util import OracleTrack, basis_as_consumed, check_close

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_a_wait_that_runs_out_is_reported_and_the_device_stays_usable():
    N, D, k, dt = 300, 1024, 64, sc.BF16
    spec = streams.StreamSpec("timeout", blocks=1, rows=N, D=D, dtype="bf16", k=k, T=2, interval=1, rank=128,
                              amp=30.0, power=1.0, noise_std=0.02)
    st = streams.BlockStream(spec, 0, device=DEV)
    basis = sc.svdcache_basis_prepare(st.V_gen[:, :k].float().contiguous(), dt)
    state = sc.new_state(N, D, k, dt, DEV)
    assert sc.svdcache_state_query(state) == (0, 0)

    sc.svdcache_selftest_wait_timeout(state, 2_000_000)      # ~1 ms at 1.9 GHz
    steps, status = sc.svdcache_state_query(state)           # synchronises the stream: the kernel has returned
    assert status == -6 and sc.lib().svdcache_status_string(status) == b"a bounded in-kernel wait ran out"
    assert steps == 0
    diag = int(state[36:40].view(torch.int32).item())        # which wait, which CTA
    assert diag == (99 << 16)
    per_warp = state[64:64 + 32].view(torch.int32).cpu().tolist()   # two warps waited: site word, progress counters
    assert per_warp[0] == diag and per_warp[4] == diag and per_warp[5] == 1

    # argument checks of the entry point itself
    L = sc.lib()
    assert L.svdcache_selftest_wait_timeout(None, 1000, None) == -1
    assert L.svdcache_selftest_wait_timeout(state.data_ptr(), 0, None) == -1
    assert L.svdcache_selftest_wait_timeout(state.data_ptr(), 10**12, None) == -1

    # the sticky status goes with a reset, and ordinary calls on the same device still work
    sc.svdcache_state_reset(state, N, D, k, dt)
    assert sc.svdcache_state_query(state) == (0, 0)
    F = st.features(0)
    out = torch.empty(N, D, dtype=torch.bfloat16, device=DEV)
    sc.svdcache_full_step(F, basis, state, k, 0.9)
    sc.svdcache_cached_step(state, basis, out, k)
    track = OracleTrack(basis_as_consumed(basis, D, k, dt), 0.9)
    Fh = F.double().cpu().numpy()
    track.full(Fh)
    check_close("Fhat", out, track.cached(), dt, float(np.sqrt(np.mean(Fh * Fh))))
    assert sc.svdcache_state_query(state) == (1, 0)
