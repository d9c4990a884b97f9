"""GPU test of co3_moments_static, the entry point for callers that may not allocate device
memory (their memory belongs to a host application's pool, or they cannot take the device-wide
synchronisation of an allocation) and so cannot create a plan.  Its result is compared with what
the regular path reports for the same inputs (co3_encode + co3_get_fit), on two calls in a row.
Collected last on purpose: a run that stops at the first failure has then run everything else."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def test_static_moments_match_the_planned_path_twice():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2203_09044_b200 import binding, inputs
    binding.lib()
    U, d, gamma = 3, 40_000, 0.9                       # d % 4 == 0 so the rows can be passed back to back
    wl = inputs.workload(0, d=d, n_users=U)
    plan = binding.Plan(d, U, 4, 3, gamma=gamma)
    assert plan.ld == d
    out = plan.alloc_outputs()
    residual = torch.zeros((U, d), device="cuda")
    moments = torch.zeros(4, dtype=torch.float64, device="cuda")
    for t in range(2):                                 # second call: non-zero memory, scratch already used
        g = wl.gradient(t, device="cuda")
        if t == 1:
            g[0, 5] = float("inf")                     # counted, left out of the sums
        m_prev = residual.clone()
        rc = binding.moments_static(g, m_prev, U * d, gamma, moments)
        assert rc == binding.OK
        torch.cuda.synchronize()
        got = moments.cpu().numpy().copy()
        rc = binding.moments_static(g, m_prev, U * d, gamma, moments)      # same inputs: same bits
        assert rc == binding.OK
        torch.cuda.synchronize()
        assert np.array_equal(got, moments.cpu().numpy())
        plan.encode(g, residual, out)                  # regular path on the same a = g + gamma m
        beta, alpha, N, S1, S2 = plan.get_fit(0)
        assert got[0] == N and got[3] == (1.0 if t == 1 else 0.0)
        np.testing.assert_allclose(got[1:3], [S1, S2], rtol=1e-12)         # the tolerance of the parity tests
    plan.status(clear=True)


def test_static_moments_refuse_what_does_not_fit():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2203_09044_b200 import binding
    binding.lib()
    g = torch.zeros(1024, device="cuda")
    moments = torch.zeros(4, dtype=torch.float64, device="cuda")
    assert binding.moments_static(g, g, binding.STATIC_MAX_ELEMENTS + 1, 0.9, moments) == binding.ELIMIT
    assert binding.moments_static(g, g, 0, 0.9, moments) == binding.EINVAL
    assert binding.moments_static(g, g, 1001, 1.0, moments) == binding.OK   # ragged tail
    torch.cuda.synchronize()
    assert moments.cpu().tolist() == [1001.0, 0.0, 0.0, 0.0]
    assert b"scratch" in binding.lib().co3_strerror(binding.ELIMIT)
