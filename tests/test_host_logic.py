"""The library's host-side logic, run without a GPU: its router against the oracle's routing simulator
(bit-exact indices), its split-K planner (every tile of every run covered exactly once), its layout
arithmetic against the header's formula, and the C-ABI surface."""
import ctypes as C
import os
import re
import subprocess

import numpy as np
import pytest

from oracle import c_oracle, np_oracle
from paper_2609_14507_b200 import binding
from tests import host_shim
from tests.conftest import ROOT


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2609_14507_b200 import build
    build.build()


def test_router_matches_oracle_on_random_programs():
    rng = np.random.default_rng(31)
    for trial in range(60):
        block = int(rng.choice([1, 4, 16, 64]))
        D = block * int(rng.integers(1, 5))
        den = int(rng.integers(1, 16)); num = int(rng.integers(0, den + 1))
        ours, ref = host_shim.Router(block, D, num, den), c_oracle.Route(block, D, num, den)
        n0 = int(rng.integers(0, 400)); den0 = int(rng.integers(1, 11)); num0 = int(rng.integers(0, den0 + 1))
        ours.bulk(n0, num0, den0); ref.bulk(n0, num0, den0)
        for _ in range(int(rng.integers(0, 600))):
            op = rng.integers(0, 40)
            if op == 0:
                ours.flush(); ref.flush()
            elif op == 1:
                s = int(rng.integers(0, den + 1)); ours.set_share(s); ref.set_share(s)
            else:
                ours.append(); ref.append()
        for a, b in zip(ours.dump(), ref.dump()):
            np.testing.assert_array_equal(a, b)
        assert ours.counts() == ref.counts()


def test_router_matches_oracle_on_paper_shaped_runs():
    # D = 256, block 64, prefill 2048 (the paper's 2K prompt), decode to 8K at the shares of Table 3
    for num, den, num0, den0 in [(15, 32, 15, 32), (35, 64, 1, 2), (5, 8, 0, 1), (0, 1, 1, 4), (1, 1, 1, 1)]:
        ours, ref = host_shim.Router(64, 256, num, den), np_oracle.Route(64, 256, num, den)
        ours.bulk(2048, num0, den0); ref.bulk(2048, num0, den0)
        for _ in range(6144 + 1):
            ours.append(); ref.append()
        for a, b in zip(ours.dump(), ref.dump()):
            np.testing.assert_array_equal(a, b)
        assert ours.counts() == ref.counts()


def test_plan_covers_every_tile_exactly_once():
    rng = np.random.default_rng(32)
    for trial in range(60):
        n_rows = int(rng.integers(1, 20))
        rows = [[int(x) for x in rng.integers(0, 5000, size=rng.integers(0, 4))] for _ in range(n_rows)]
        n_gh = int(rng.choice([1, 4, 8]))
        splits = int(rng.choice([0, 0, 1, 3, 16]))
        cps = int(rng.choice([1, 2]))
        p = host_shim.plan(rows, n_gh, splits, cps)
        live = [[n for n in row if n > 0] for row in rows]
        assert list(p["seg_tokens"]) == [n for row in live for n in row]
        n_spans = len(p["row"])
        css, rgs = p["cta_span_start"], p["rg_span_start"]
        assert css[0] == 0 and css[-1] == n_spans and np.all(np.diff(css) >= 0) and len(css) - 1 <= 148 * cps
        assert rgs[0] == 0 and rgs[-1] == n_spans and np.all(np.diff(rgs) >= 0)
        assert np.all(p["ntiles"] >= 1)
        # tiles per chunk, the table the dynamically balanced kernel looks for work in
        assert list(p["cta_tiles"]) == [int(p["ntiles"][css[c]:css[c + 1]].sum()) for c in range(len(css) - 1)]
        assert p["table_bytes"] > 0
        seg_id0 = 0
        for r, row in enumerate(live):
            for gh in range(n_gh):
                k0, k1 = rgs[r * n_gh + gh], rgs[r * n_gh + gh + 1]
                assert np.all(p["row"][k0:k1] == r) and np.all(p["gh"][k0:k1] == gh)
                covered = {}
                for k in range(k0, k1):
                    covered.setdefault(int(p["seg"][k]), []).append((int(p["tile0"][k]), int(p["ntiles"][k])))
                for j, n in enumerate(row):
                    t = 0
                    for t0, cnt in sorted(covered.pop(seg_id0 + j)):
                        assert t0 == t
                        t += cnt
                    assert t == -(-n // 64)
                assert not covered
            seg_id0 += len(row)
        # every CTA gets the same number of tiles (within one) when the planner balances freely
        loads = np.array([p["ntiles"][css[c]:css[c + 1]].sum() for c in range(len(css) - 1)])
        if loads.size:
            assert loads.sum() == p["ntiles"].sum()
            assert loads.max() - loads.min() <= 1, (loads.min(), loads.max(), splits)


def test_plan_fills_the_machine_in_one_balanced_wave():
    # Qwen3-shaped step: 16 rows x (32512 resident + 257 window tokens), 4 KV heads: 296 CTAs, equal loads
    p = host_shim.plan([[32768 - 256, 257]] * 16, 4)
    css = p["cta_span_start"]
    assert len(css) - 1 == 296
    loads = np.array([p["ntiles"][css[c]:css[c + 1]].sum() for c in range(296)])
    assert loads.max() - loads.min() <= 1 and loads.sum() == 16 * 4 * (508 + 5)
    # few spans: one cut per CTA boundary plus one per (row, head, run)
    assert len(p["row"]) <= 296 + 16 * 4 * 2
    # a tiny launch uses as many CTAs as it has tiles
    p = host_shim.plan([[100], [1]], 4)
    assert len(p["cta_span_start"]) - 1 == 4 * (2 + 1)


def test_span_bound_and_scratch_size_hold_for_ragged_rows_with_explicit_splits():
    """With kv_splits the planner first cuts every row into pieces and then cuts pieces again where a CTA's chunk ends;
    ragged rows make those second cuts fall inside pieces.  The span bound (checked inside the shim) and the scratch
    size the library reports must cover the plan that is actually built."""
    from paper_2609_14507_b200 import binding
    shapes = [(binding.GQA, 32, 4, 128, 128, 4, 8, 4, 2), (binding.MLA, 16, 1, 576, 512, 1, 16, 1, 1)]
    cases = [[32768 - 192 * i for i in range(16)], [6400, 6208], [70000, 69000, 50, 1], [4096] * 40 + [33]]
    for kind, hq, hkv, dqk, dv, n_gh, rows_per_group, parts, cps in shapes:
        shape = binding.make_shape(kind, hq, hkv, dqk, dv, 64, 0.0)
        for lens in cases:
            for splits in (2, 4, 8, 64):
                rows = [[n] for n in lens]
                p = host_shim.plan(rows, n_gh, splits, cps)           # raises if the bound is exceeded
                n_spans = len(p["row"])
                part_rows = n_spans * parts * rows_per_group
                need = -(-p["table_bytes"] // 256) * 256 + 256 + -(-part_rows * dv * 4 // 256) * 256 + -(-part_rows * 4 // 256) * 256
                got = binding.ipkv_attend_scratch_bytes(shape, len(rows), len(rows), sum(lens), splits)
                assert need <= got, (kind, lens[:2], splits, n_spans, need, got)


def test_balancing_threshold_follows_the_measured_crossovers():
    """The rule that decides when the grouped-query kernel balances its load: 64 tiles per CTA while the split reduce
    fits one wave of CTAs, more for larger batches (the two measured cross-overs: 60-70 tiles per CTA for 16 rows x
    32 heads, about 135 for 64 rows x 32 heads); monotone in the batch."""
    f = host_shim.lib().shim_min_tiles_to_balance
    assert f(16, 32) == 64 and f(1, 8) == 64 and f(18, 32) == 64
    assert 125 <= f(64, 32) <= 140
    vals = [f(r, 32) for r in range(1, 400, 7)]
    assert vals == sorted(vals)


def test_layout_arithmetic_matches_header_formula():
    L = host_shim.lib()
    for bt in (16, 64, 256):
        for t in range(bt):
            for chunk in range(72):
                x = chunk * 8
                want = (x // 64) * bt * 128 + t * 128 + ((((x % 64) // 8) ^ (t & 7)) * 16)
                assert L.shim_tile_chunk_offset(bt, t, chunk) == want
                assert L.shim_plain_chunk_offset(576, t, chunk) == (t * 576 + x) * 2
    # bytes per token per layer: the sizes behind Tables 1 and 2
    assert L.shim_block_bytes(4, 128, 128, 64) == 64 * 2048
    assert L.shim_block_bytes(8, 128, 128, 64) == 64 * 4096
    assert L.shim_block_bytes(1, 576, 0, 64) == 64 * 1152


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "ipkv.h")).read()
    declared = sorted(set(re.findall(r"\b(ipkv_[a-z_]+)\s*\(", header)))
    assert declared and set(declared) == set(binding.EXPORTS)
    L = binding.lib()
    for name in declared:
        assert hasattr(L, name), name


def test_struct_sizes_match_the_c_header(tmp_path):
    src = tmp_path / "sz.c"
    src.write_text('#include <stdio.h>\n#include "ipkv.h"\nint main(void){printf("%zu %zu %zu %zu %zu %zu\\n", sizeof(ipkv_config),'
                   'sizeof(ipkv_attend_opts), sizeof(ipkv_extent), sizeof(ipkv_stats), sizeof(ipkv_attn_shape), sizeof(ipkv_run));return 0;}\n')
    exe = tmp_path / "sz"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    sizes = [int(x) for x in subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.split()]
    assert sizes == [C.sizeof(binding.Config), C.sizeof(binding.AttendOpts), C.sizeof(binding.Extent),
                     C.sizeof(binding.Stats), C.sizeof(binding.AttnShape), C.sizeof(binding.Run)]


def test_query_sizes_reproduce_table2(golden):
    # The library's own sizing of W and PP (no GPU needed) against Table 2: bs=32, D=256, two
    # ping-pong slots of 512 tokens per sequence.
    shapes = {"ds2": (binding.MLA, 27, 16, 1, 576, 512), "qwen3": (binding.GQA, 48, 32, 4, 128, 128),
              "mixtral": (binding.GQA, 32, 32, 8, 128, 128)}
    for name, (kind, nl, hq, hkv, dqk, dv) in shapes.items():
        cfg = binding.make_config(kind, nl, 32, hq, hkv, dqk, dv, block_tokens=64, window_tokens=256, chunk_tokens=512,
                                  n_slots=2, max_u_tokens_per_seq=0, max_p_tokens_per_seq=0)
        s = binding.ipkv_query_sizes(cfg)
        assert abs(s["w"] / 1e6 - golden[f"table2.dwindow_mb.{name}"]) < 0.5
        assert abs(s["pp"] / 1e6 - golden[f"table2.pingpong_mb.{name}"]) < 0.06
        assert s["resident"] == 0 and s["u"] == 0 and s["p"] == 0


def test_bad_configs_are_rejected_and_no_gpu_fails_loudly():
    good = dict(block_tokens=64, window_tokens=256, chunk_tokens=512)
    for kw in (dict(block_tokens=48), dict(window_tokens=100), dict(chunk_tokens=96), dict(n_slots=1),
               dict(share_num=3, share_den=2), dict(share_den=0)):
        cfg = binding.make_config(binding.GQA, 1, 1, 32, 4, 128, 128, **{**good, **kw})
        with pytest.raises(binding.IpkvError):
            binding.ipkv_query_sizes(cfg)
    for dims in ((32, 5, 128, 128), (32, 4, 96, 96), (32, 4, 128, 64)):
        cfg = binding.make_config(binding.GQA, 1, 1, *dims, **good)
        with pytest.raises(binding.IpkvError):
            binding.ipkv_query_sizes(cfg)
    import torch
    if not torch.cuda.is_available():
        cfg = binding.make_config(binding.GQA, 1, 1, 32, 4, 128, 128, **good)
        with pytest.raises(binding.IpkvError) as e:
            binding.Cache(cfg)
        assert e.value.status == 5          # IPKV_ECUDA: no silent CPU path


def test_device_status_word_maps_to_the_documented_messages():
    """Bits of the device status word (which bounded wait of a kernel gave up) -> the text behind IPKV_ETIMEOUT."""
    import ctypes
    L = host_shim.lib()
    L.shim_status_bit.restype = ctypes.c_uint32
    bits = [L.shim_status_bit(i) for i in range(3)]
    assert bits == [1, 2, 4]                      # the values include/ipkv.h documents for ipkv_stats.device_status

    def text(word):
        buf = ctypes.create_string_buffer(256)
        assert L.shim_describe_status(ctypes.c_uint32(word), buf, 256) >= 0
        return buf.value.decode()

    assert text(0) == ""
    assert "free stage" in text(1) and "tile" not in text(1)
    assert "no tile" in text(2) and "free stage" not in text(2)
    assert "did not land" in text(4)
    assert all(k in text(7) for k in ("free stage", "no tile", "did not land"))
    assert "left its region" in text(8) and "unknown" in text(16)


def test_resident_ring_never_hands_a_slot_out_twice():
    """Per-sequence ring capacities: the slots of all blocks that are resident at the same time (the newest cap[s] P
    blocks of every sequence) are distinct and inside the layer's ring, whatever the capacities and fill levels; a
    uniform capacity is the special case; the sizes the library reports follow the capacities."""
    import ctypes
    from paper_2609_14507_b200 import binding
    L = host_shim.lib()
    L.shim_ring_slots.restype = ctypes.c_int64
    vp, i64 = ctypes.c_void_p, ctypes.c_int64
    L.shim_ring_slots.argtypes = [ctypes.c_int, i64, vp, i64, vp, vp, i64, ctypes.POINTER(i64), vp]
    rng = np.random.default_rng(51)
    for trial in range(200):
        n = int(rng.integers(1, 40))
        bt = int(rng.choice([16, 32, 64, 128]))
        by_seq = rng.integers(0, 3000, size=n).astype(np.int64) if trial % 3 else None
        uniform = int(rng.integers(0, 3000))
        used = rng.integers(0, 120, size=n).astype(np.int64)
        out = np.zeros(200000, dtype=np.int64); caps = np.zeros(n, dtype=np.int64); total = ctypes.c_int64()
        k = L.shim_ring_slots(n, uniform, by_seq.ctypes.data if by_seq is not None else None, bt,
                              used.ctypes.data, out.ctypes.data, out.size, ctypes.byref(total), caps.ctypes.data)
        assert k >= 0
        want_caps = [-(-int(t) // bt) for t in (by_seq if by_seq is not None else [uniform] * n)]
        assert list(caps) == want_caps and total.value == sum(want_caps)
        slots = out[:k]
        assert k == sum(min(int(u), c) for u, c in zip(used, want_caps))
        assert len(set(slots.tolist())) == k                              # no slot twice
        assert k == 0 or (slots.min() >= 0 and slots.max() < total.value)
    # the sizes: every layer's ring is the sum of the sequences' capacities
    lens = [100, 6400, 0, 777]
    cfg = binding.make_config(binding.GQA, 3, 4, 32, 4, 128, 128, block_tokens=64, window_tokens=256, chunk_tokens=512,
                              max_u_tokens_per_seq=64, max_p_tokens_per_seq=8192, resident_tokens_per_seq=8192,
                              resident_tokens_by_seq=lens, flags=binding.FLAG_NO_HOST_U | binding.FLAG_NO_HOST_P)
    sizes = binding.ipkv_query_sizes(cfg)
    assert sizes["resident"] == 3 * sum(-(-x // 64) for x in lens) * 64 * 2048
    cfg_u = binding.make_config(binding.GQA, 3, 4, 32, 4, 128, 128, block_tokens=64, window_tokens=256, chunk_tokens=512,
                                max_u_tokens_per_seq=64, max_p_tokens_per_seq=8192, resident_tokens_per_seq=8192,
                                flags=binding.FLAG_NO_HOST_U | binding.FLAG_NO_HOST_P)
    assert binding.ipkv_query_sizes(cfg_u)["resident"] == 3 * 4 * 128 * 64 * 2048


def test_window_fill_travels_as_a_launch_parameter_while_the_batch_is_in_lockstep():
    """When every D-window run of a launch ends at the same offset inside its last 64-token tile, the runs are stored
    rounded up to whole tiles and the offset becomes the launch parameter: two consecutive decode steps then have
    byte-identical tables (no upload), until the windows grow into a new tile.  Windows that disagree keep their exact
    counts in the table (parameter 0), and the tables differ from step to step."""
    import ctypes
    L = host_shim.lib()
    i64 = ctypes.c_int64

    def two_steps(resident, fills, n_gh=4, cps=2):
        res = (i64 * len(resident))(*resident); fl = (i64 * len(fills))(*fills)
        same, nxt = ctypes.c_int(), ctypes.c_int()
        t = L.shim_window_tail(len(resident), res, fl, n_gh, cps, ctypes.byref(same), ctypes.byref(nxt))
        return t, nxt.value, bool(same.value)

    assert two_steps([8192] * 4, [5] * 4) == (5, 6, True)
    assert two_steps([8192, 100, 33000], [63, 127, 191]) == (63, 64, True)     # different windows, same offset in the last tile
    assert two_steps([8192] * 4, [64] * 4) == (64, 1, False)                   # the next token opens a new tile: a new plan
    assert two_steps([8192] * 4, [0] * 4)[0] == 0                              # no window tokens yet: nothing to flag
    t, nxt, same = two_steps([8192, 8192], [5, 6])
    assert (t, nxt, same) == (0, 0, False)                                     # windows out of step: exact counts, tables differ
    assert two_steps([0, 8192], [17, 17], n_gh=1, cps=1) == (17, 18, True)     # a row with nothing but its window


def test_consumer_warps_join_their_partials_only_in_launches_with_long_spans():
    """The grouped-query kernel writes one partial per span (its four warps join their states first) when the launch's
    spans are long, four when they are short; the compressed-latent kernel always writes one."""
    L = host_shim.lib()
    i64 = C.c_int64
    L.shim_parts_per_span.restype = C.c_int
    L.shim_parts_per_span.argtypes = [C.c_int, C.c_int, C.POINTER(i64), C.c_int, C.c_int]

    def parts(kind, tokens, n_gh, cps):
        return L.shim_parts_per_span(kind, len(tokens), (i64 * len(tokens))(*tokens), n_gh, cps)

    assert parts(0, [24577] * 16, 8, 2) == 1            # Mixtral shape at a quarter on the CPU: 116 tiles per span
    assert parts(0, [32769] * 16, 4, 2) == 1            # Qwen3 shape, everything on the GPU
    assert parts(0, [9831] * 16, 4, 2) == 1             # the same at 70 % on the CPU: 24 tiles per span, but 1.2 spans per CTA
    assert parts(0, [4097], 4, 2) == 4                  # one short sequence: one tile per CTA
    assert parts(0, [100, 1], 4, 2) == 4
    assert parts(1, [78644] * 8, 1, 1) == 1 and parts(1, [100], 1, 1) == 1
    # the rule itself on the launches it was measured on: (tiles, spans, CTAs)
    L.shim_parts_rule.restype = C.c_int
    L.shim_parts_rule.argtypes = [C.c_int, i64, i64, i64]
    rule = lambda tiles, spans, ctas: L.shim_parts_rule(0, tiles, spans, ctas)
    assert rule(65600, 808, 296) == 1 and rule(46000, 808, 296) == 1        # ragged batch of 64, CPU share 0 and 30 %: long spans
    assert rule(32800, 808, 296) == 4 and rule(19700, 808, 296) == 4        # at 50 and 70 %: 41 and 24 tiles per span, 2.7 spans per CTA
    assert rule(6600, 808, 296) == 4                                        # at 90 %
    assert rule(9856, 424, 296) == 1                                        # Qwen3 shape at 70 %: 23 tiles per span, 1.4 spans per CTA
    assert rule(260, 264, 260) == 4                                         # one 4K sequence: single-tile spans
    assert rule(0, 0, 0) == 4
