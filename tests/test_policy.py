"""Roofline share model and policy (Sec. 5.2-5.3): the oracle's formulas against the algebra the paper fixes, and the
library's host-side policy (no GPU involved) against the oracle."""
import numpy as np
import pytest

from oracle import c_oracle, np_oracle
from paper_2609_14507_b200 import binding


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2609_14507_b200 import build
    build.build()


MODELS = [dict(A=4e-9, B=4e-9, C_cpu=2e-4, C_gpu=5e-4),       # A = B, positive Delta (the DeepSeek-V2-Lite picture)
          dict(A=9e-9, B=4e-9, C_cpu=6e-4, C_gpu=1e-4),       # negative Delta (the Qwen3 picture)
          dict(A=1e-9, B=40e-9, C_cpu=0.0, C_gpu=0.0),
          dict(A=50e-9, B=1e-9, C_cpu=1e-3, C_gpu=0.0)]


def test_eq2_balances_eq1_where_it_is_not_clamped():
    # Eq. 2 is the solution of T_CPU(r) = T_GPU(r): check it by evaluating Eq. 1 at the returned share.
    for m in MODELS:
        for L in (512, 2048, 8192, 32768, 1 << 20):
            r = np_oracle.roofline_share(L=L, **m)
            tc, tg = np_oracle.engine_times(r=r, L=L, **m)
            if 0.0 < r < 1.0:
                assert tc == pytest.approx(tg, rel=1e-12)
            elif r == 0.0:
                assert tc <= tg + 1e-15 or m["C_cpu"] >= tg     # the CPU side is already the slower one with no tokens
            else:
                assert tg <= tc + 1e-15 or m["C_gpu"] >= tc
            # no other share does better than the balanced one (T is the max of a rising and a falling line)
            best = max(tc, tg)
            for rr in np.linspace(0, 1, 201):
                a, b = np_oracle.engine_times(r=rr, L=L, **m)
                assert max(a, b) >= best - 1e-15


def test_eq2_limits_and_clamps():
    m = MODELS[0]
    # A = B: the share decays from above to the converged value 0.50 as L grows (positive Delta), Sec. 5.3
    shares = [np_oracle.roofline_share(L=L, **m) for L in (1 << 17, 1 << 20, 1 << 24, 1 << 30)]
    assert shares == sorted(shares, reverse=True) and shares[-1] == pytest.approx(0.5, abs=1e-4) and 1.0 > shares[0] > 0.5
    m = MODELS[1]
    shares = [np_oracle.roofline_share(L=L, **m) for L in (1 << 17, 1 << 20, 1 << 24, 1 << 30)]
    assert shares == sorted(shares) and shares[-1] == pytest.approx(4 / 13, abs=1e-4) and shares[0] > 0.0   # rises to B/(A+B)
    assert np_oracle.roofline_share(A=1e-9, B=1e-9, C_cpu=1.0, C_gpu=0.0, L=100) == 0.0     # clamps
    assert np_oracle.roofline_share(A=1e-9, B=1e-9, C_cpu=0.0, C_gpu=1.0, L=100) == 1.0


def test_library_model_matches_oracle():
    for m in MODELS:
        for L in (1, 512, 4096, 131072):
            assert binding.ipkv_roofline_share(L=L, **m) == pytest.approx(np_oracle.roofline_share(L=L, **m), rel=1e-14, abs=1e-16)
            for r in (0.0, 0.3, 1.0):
                t, tc, tg = binding.ipkv_roofline_step_time(r=r, L=L, t_merge=5e-4, **m)
                otc, otg = np_oracle.engine_times(r=r, L=L, **m)
                assert (tc, tg) == pytest.approx((otc, otg), rel=1e-14)
                assert t == pytest.approx(max(otc, otg) + 5e-4, rel=1e-14)
    assert np.isnan(binding.ipkv_roofline_share(A=0.0, B=1.0, C_cpu=0, C_gpu=0, L=10))


def test_feedback_recovers_the_cpu_cost_and_steers_the_router():
    # The CPU engine's true cost drifts from the calibrated 4 ns to 12 ns per token; after a window of noisy step
    # latencies the policy's estimate follows, and the marginal share moves from 1/2 to B/(A+B) = 1/4.
    rng = np.random.default_rng(81)
    true_A, B, C_cpu = 12e-9, 4e-9, 3e-4
    pol = binding.Policy(A=4e-9, B=B, C_cpu=C_cpu, C_gpu=1e-4, window_steps=256, share_den=64)
    num, model = pol.update()
    assert num == 32 and model["A"] == 4e-9                   # no samples yet: calibrated value
    lat, toks = [], []
    for step in range(600):
        n_cpu = 16 * (8192 + 3 * step)                          # CPU-side tokens grow with the decode
        t = true_A * n_cpu + C_cpu + rng.normal(0.0, 2e-5)
        pol.observe(t, n_cpu)
        lat.append(t); toks.append(n_cpu)
    num, model = pol.update()
    want_A = np_oracle.estimate_A(lat[-256:], toks[-256:], C_cpu)
    assert model["A"] == pytest.approx(want_A, rel=1e-9)
    assert model["A"] == pytest.approx(true_A, rel=0.01)
    assert num == round(64 * B / (want_A + B)) == 16
    # prefill share R(L0) = r(L0), quantised to the denominator
    assert pol.prefill_share(2048) == round(64 * np_oracle.roofline_share(A=model["A"], B=B, C_cpu=C_cpu, C_gpu=1e-4, L=2048))
    # fed to the router, the cumulative share follows R(L) = p + (R(L0) - p) L0 / L within half a batch (Sec. 5.3)
    D, L0 = 256, 2048
    r = c_oracle.Route(64, D, num, 64)
    r.bulk(L0, pol.prefill_share(L0), 64)
    R0 = r.counts()["n_u"] / L0
    for _ in range(40 * D + 1):
        r.append()
    c = r.counts()
    L = c["n_u"] + c["n_p"]
    assert abs(c["n_u"] / L - np_oracle.cumulative_share(num / 64, R0, L0, L)) <= D / (2 * L) + 1e-12


def test_policy_rejects_bad_input():
    with pytest.raises(binding.IpkvError):
        binding.Policy(A=-1.0, B=1.0, C_cpu=0, C_gpu=0)
    pol = binding.Policy(A=1e-9, B=1e-9, C_cpu=0, C_gpu=0)
    with pytest.raises(binding.IpkvError):
        pol.observe(float("nan"), 10)
