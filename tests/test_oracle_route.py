"""Pins for the routing oracle (O3): conservation, immutability, the closed forms of Sec. 5.3,
the clamps, the region sizes of Tables 1-2 and the batch quantisation visible in Table 3."""
import itertools

import numpy as np
import pytest

from oracle import c_oracle, np_oracle

ROUTES = [pytest.param(c_oracle.Route, id="cpp"), pytest.param(np_oracle.Route, id="numpy")]
U, P, W = 0, 1, 2


def closed_form(block, D, num, den, n0, num0, den0, steps):
    """Independent restatement: where every token ends up after a prefill of n0 tokens and
    ``steps`` lazily-flushed decode appends at a constant share num/den.

    Batch j (1-based) is CPU-placed iff round-half-up(j*p) exceeds round-half-up((j-1)*p)."""
    n = n0 + steps
    region = np.empty(n, np.int8); blk = np.empty(n, np.int64); off = np.empty(n, np.int32)
    n_cpu = block * ((n0 // block) * num0 // den0)
    t = np.arange(n0)
    region[:n_cpu] = U; region[n_cpu:n0] = P
    blk[:n_cpu] = t[:n_cpu] // block; off[:n_cpu] = t[:n_cpu] % block
    blk[n_cpu:n0] = (t[n_cpu:] - n_cpu) // block; off[n_cpu:n0] = (t[n_cpu:] - n_cpu) % block
    nb = {U: n_cpu // block, P: -(-(n0 - n_cpu) // block)}
    n_batches = max(0, (steps - 1) // D) if steps > 0 else 0      # full windows already evicted
    hup = lambda j: (j * num + den // 2) // den
    for j in range(1, n_batches + 1):
        dest = U if hup(j) > hup(j - 1) else P
        first = n0 + (j - 1) * D
        tt = np.arange(D)
        region[first:first + D] = dest
        blk[first:first + D] = nb[dest] + tt // block
        off[first:first + D] = tt % block
        nb[dest] += D // block
    w_first = n0 + n_batches * D
    region[w_first:] = W; blk[w_first:] = 0; off[w_first:] = np.arange(n - w_first)
    return region, blk, off, hup(n_batches), n_batches


@pytest.mark.parametrize("Route", ROUTES)
def test_exhaustive_small_grid_matches_closed_form(Route):
    for block, mult, n0, (num, den), (num0, den0), steps in itertools.product(
            (1, 2, 4), (1, 2, 3), (0, 1, 5, 8, 13), ((0, 1), (1, 1), (1, 2), (1, 3), (3, 8), (5, 7)),
            ((0, 1), (1, 2), (1, 1), (2, 5)), (0, 1, 4, 9, 25)):
        D = block * mult
        r = Route(block, D, num, den)
        r.bulk(n0, num0, den0)
        for _ in range(steps):
            r.append()
        region, blk, off = r.dump()
        e_region, e_blk, e_off, n_cpu_batches, n_batches = closed_form(block, D, num, den, n0, num0, den0, steps)
        ctx = (block, D, n0, num, den, num0, den0, steps)
        np.testing.assert_array_equal(region, e_region, err_msg=str(ctx))
        np.testing.assert_array_equal(blk, e_blk, err_msg=str(ctx))
        np.testing.assert_array_equal(off, e_off, err_msg=str(ctx))
        c = r.counts()
        assert c["n_flush"] == n_batches and c["n_flush_cpu"] == n_cpu_batches, ctx


@pytest.mark.parametrize("Route", ROUTES)
def test_conservation_window_bounds_and_immutability(Route):
    rng = np.random.default_rng(21)
    block, D = 4, 12
    r = Route(block, D, 3, 7)
    r.bulk(30, 2, 5)
    seen = {}
    for step in range(200):
        op = rng.integers(0, 20)
        if op == 0:
            r.flush()                               # explicit (possibly partial) eviction
        elif op == 1:
            r.set_share(int(rng.integers(0, 8)))
        else:
            r.append()
            c = r.counts()
            assert 1 <= c["n_w"] <= D               # the newest token is always GPU-side
        region, blk, off = r.dump()
        c = r.counts()
        assert c["n_u"] + c["n_p"] + c["n_w"] == len(r) == len(region)
        # every placed location is unique inside its region, and never changes once placed
        for reg in (U, P):
            loc = [(int(b), int(o)) for g, b, o in zip(region, blk, off) if g == reg]
            assert len(loc) == len(set(loc))
            assert all(0 <= o < block for _, o in loc)
        for t, (g, b, o) in enumerate(zip(region, blk, off)):
            if g != W:
                if t in seen:
                    assert seen[t] == (g, b, o)
                seen[t] = (g, b, o)
        # batches are whole and start on a block boundary: offset 0 wherever the region or run changes
        for t in range(1, len(region)):
            if region[t] != W and region[t] != region[t - 1]:
                assert off[t] == 0


@pytest.mark.parametrize("Route", ROUTES)
def test_share_clamps(Route):
    r = Route(16, 64, 0, 1)
    r.bulk(128, 1, 2)
    for _ in range(64 * 5 + 1):
        r.append()
    c = r.counts()
    assert c["n_u"] == 64 and c["n_flush_cpu"] == 0 and c["n_p"] == 64 + 64 * 5
    r = Route(16, 64, 1, 1)
    r.bulk(128, 0, 1)
    for _ in range(64 * 5 + 1):
        r.append()
    c = r.counts()
    assert c["n_p"] == 128 and c["n_u"] == 64 * 5 and c["n_flush_cpu"] == 5


@pytest.mark.parametrize("Route", ROUTES)
def test_cumulative_share_tracks_closed_form(Route):
    # Sec. 5.3: R(L) = p + (R(L0) - p) * L0 / L, moving by D/L per batch; the integer rule stays within
    # half a batch of it.
    block, D, L0 = 64, 256, 2048
    for (num, den), (num0, den0) in [((1, 2), (1, 4)), ((5, 8), (0, 1)), ((3, 10), (9, 10)), ((1, 3), (1, 3))]:
        r = Route(block, D, num, den)
        r.bulk(L0, num0, den0)
        R0 = r.counts()["n_u"] / L0
        p = num / den
        for _ in range(120 * D + 1):              # the 120th batch leaves the window at the last append
            r.append()
        c = r.counts()
        L = c["n_u"] + c["n_p"]
        assert L == L0 + 120 * D
        target = p * L + (R0 - p) * L0            # = R(L) * L
        assert abs(c["n_u"] - target) <= D / 2 + 1e-9
        assert abs(c["n_u"] / L - (p + (R0 - p) * L0 / L)) <= D / (2 * L) + 1e-12


@pytest.mark.parametrize("Route", ROUTES)
def test_table3_shares_are_whole_batches(Route, golden):
    # Table 3: the solo shares are multiples of D/L with D = 256 (0.469 = 15/32 at 8K, 0.438 = 14/32,
    # 0.547 = 35/64 at 16K); the router reaches each of them exactly from an empty prefill share.
    D, block = 256, 64
    for key, L, batches in [("table3.solo_r.bs8_8k", 8192, 15), ("table3.solo_r.bs4_8k", 8192, 14),
                            ("table3.solo_r.bs16_16k", 16384, 35), ("table3.adaptive_r.bs8_8k_low", 8192, 12)]:
        n_batches = L // D
        assert round(batches / n_batches, 3) == golden[key]
        r = Route(block, D, batches, n_batches)
        r.bulk(0, 0, 1)
        for _ in range(L + 1):
            r.append()
        c = r.counts()
        assert c["n_u"] + c["n_p"] == L and c["n_u"] == batches * D
    assert 5 / 8 == golden["sec2_2.max_share.qwen3"]
    assert 256 / 2048 == golden["sec7_6.batch_fraction_2k"]
    assert golden["sec5_3.max_share_deviation"] <= 0.5 * golden["sec7_6.batch_fraction_2k"]


def test_bytes_per_token_and_footprint_reproduce_tables(golden):
    shapes = {"ds2": ("mla", 1, 576, 512, 27), "qwen3": ("gqa", 4, 128, 128, 48), "mixtral": ("gqa", 8, 128, 128, 32)}
    for name, (kind, hkv, dqk, dv, nl) in shapes.items():
        bpt = np_oracle.kv_bytes_per_token(kind, hkv, dqk, dv)
        assert bpt == {"ds2": 1152, "qwen3": 2048, "mixtral": 4096}[name]
        # Table 1: KV at bs=4 x 32K
        assert round(bpt * nl * 4 * 32768 / 1e9, 1) == golden[f"table1.kv_gb.{name}"]
        # Table 2: bs=32 x 32K, D=256, ping-pong of 1024 tokens per sequence; U + P = full KV
        u_tokens = round(golden[f"table2.unpinned_gb.{name}"] * 1e9 / (bpt * nl * 32))
        fp = np_oracle.footprint(bpt, nl, 32, 32768, 256, 1024, u_tokens)
        assert abs(fp["pingpong"] / 1e6 - golden[f"table2.pingpong_mb.{name}"]) < 0.06
        assert abs(fp["dwindow"] / 1e6 - golden[f"table2.dwindow_mb.{name}"]) < 0.5
        assert abs(fp["pinned"] / 1e9 - golden[f"table2.pinned_gb.{name}"]) < 0.006
        assert abs((fp["unpinned"] + fp["pinned"]) / 1e9
                   - (golden[f"table2.unpinned_gb.{name}"] + golden[f"table2.pinned_gb.{name}"])) < 0.011
        assert fp["unpinned"] + fp["pinned"] == fp["full"]
        assert round((fp["pingpong"] + fp["dwindow"]) / 1e6 / 1024, 2) == golden[f"sec7_7.gpu_resident_gb.{name}"]


def test_cpp_and_numpy_routes_agree_on_random_programs():
    rng = np.random.default_rng(22)
    for trial in range(30):
        block = int(rng.choice([1, 2, 8, 16]))
        D = block * int(rng.integers(1, 5))
        den = int(rng.integers(1, 12)); num = int(rng.integers(0, den + 1))
        a, b = c_oracle.Route(block, D, num, den), np_oracle.Route(block, D, num, den)
        n0 = int(rng.integers(0, 100)); den0 = int(rng.integers(1, 9)); num0 = int(rng.integers(0, den0 + 1))
        a.bulk(n0, num0, den0); b.bulk(n0, num0, den0)
        for _ in range(int(rng.integers(0, 150))):
            op = rng.integers(0, 12)
            if op == 0:
                a.flush(); b.flush()
            elif op == 1:
                s = int(rng.integers(0, den + 1)); a.set_share(s); b.set_share(s)
            else:
                a.append(); b.append()
        for x, y in zip(a.dump(), b.dump()):
            np.testing.assert_array_equal(x, y)
        assert a.counts() == b.counts()
