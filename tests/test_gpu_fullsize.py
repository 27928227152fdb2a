"""Parity at the benchmark's sizes and launch configuration, on sampled outputs the oracle computes one by one.

The caches are built exactly as bench.py builds them (same shapes, seeds, shares, flags); one decode step is run the
way bench.py runs it (append riding in the attention call, balanced schedule, fold in the split reduce) and, for a sample of (layer, sequence) pairs, the oracle recomputes the GPU-side partial of
every head from the same bits (regenerated from the seed and copied to the host)."""
import numpy as np
import pytest

import bench
from oracle import c_oracle
from paper_2609_14507_b200 import synth
from tests.gpu_util import check_partial

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")
DEV = "cuda:0"


def _run_step_and_check(name, samples, kv_splits=0):
    wl = bench.WORKLOADS[name]
    sh, B = wl["shape"], wl["batch"]
    num0, den0 = wl["share"]
    lens = bench.seq_lens(wl)
    need = sum(n - bench.cpu_tokens(n, num0, den0) for n in lens) * sh.n_layers * sh.bytes_per_token
    free, _ = torch.cuda.mem_get_info()
    if free < 1.3 * need:
        pytest.skip(f"needs {need / 1e9:.0f} GB of device memory")
    cache = bench.make_cache(wl, 0, 8)
    try:
        bench.populate(cache, wl, DEV)
        g = torch.Generator(device=DEV); g.manual_seed(123)
        ids = list(range(B))
        scale = float(np.float32(sh.scale))
        for layer in sorted({l for l, _ in samples}):
            q = torch.randn((B, sh.n_q_heads, sh.dim_qk), generator=g, device=DEV).to(torch.bfloat16)
            kn = torch.randn((B, sh.n_kv_heads, sh.dim_qk), generator=g, device=DEV).to(torch.bfloat16)
            vn = None if sh.kind == "mla" else torch.randn((B, sh.n_kv_heads, sh.dim_v), generator=g, device=DEV).to(torch.bfloat16)
            # as bench.py issues a layer: the append rides in the attention call (written by the kernel itself for the
            # grouped-query shapes), launches this long are dynamically balanced, and a partial is folded in by the
            # split reduce (an empty one here, so that the output stays the GPU-side partial the oracle recomputes)
            o = torch.zeros((B, sh.n_q_heads, sh.dim_v), device=DEV); lse = torch.zeros((B, sh.n_q_heads), device=DEV)
            fold_o = torch.zeros((B, sh.n_q_heads, sh.dim_v), device=DEV)
            fold_lse = torch.full((B, sh.n_q_heads), float("-inf"), device=DEV)
            cache.attend_gpu(layer, ids, q, o, lse, kv_splits=kv_splits, append_k=kn, append_v=vn, fold_o=fold_o, fold_lse=fold_lse)
            torch.cuda.synchronize()
            o_h, lse_h, q_h = o.cpu().numpy(), lse.cpu().numpy(), synth.torch_bits(q)
            kn_h, vn_h = synth.torch_bits(kn), (None if vn is None else synth.torch_bits(vn))
            for (l, s) in samples:
                if l != layer:
                    continue
                n = lens[s]
                c = cache.counts(layer, s)
                n_cpu = bench.cpu_tokens(n, num0, den0)
                assert (c["n_u"], c["n_p"], c["n_w"]) == (n_cpu, n - n_cpu, 1)
                kd, vd = synth.device_kv(sh, n, bench.kv_seed(wl, layer, s), DEV)
                k = np.concatenate([synth.torch_bits(kd), kn_h[s:s + 1]])
                v = sh.dim_v if vd is None else np.concatenate([synth.torch_bits(vd), vn_h[s:s + 1]])
                o_ref, l_ref = c_oracle.attend(q_h[s], k, v, np.arange(n_cpu, n + 1), scale)
                check_partial(o_h[s], lse_h[s], o_ref, l_ref, f"{name} layer {layer} seq {s}")
                # contents of the newest token and of a few routed ones, bit for bit
                for t in (n, n - 1, n_cpu, (n_cpu + n) // 2):
                    kk, vv = cache.read_token(layer, s, t)
                    np.testing.assert_array_equal(kk, k[t])
                    if vv is not None:
                        np.testing.assert_array_equal(vv, v[t])
        stats = cache.get_stats()
        assert stats["device_status"] == 0
        return stats
    finally:
        cache.close()
        torch.cuda.empty_cache()


def test_mixtral_32k_bench_configuration():
    _run_step_and_check("mixtral-8x7b-bs16-32k-cpu25", [(0, 0), (0, 15), (17, 6), (31, 9)])


def test_qwen3_32k_share_sweep_sampled():
    for name in ("qwen3-2layers-bs16-32k-cpu0",):
        _run_step_and_check(name, [(0, 3), (1, 12)])
    for num in (1, 3, 5, 7):                              # CPU share 10 / 30 / 50 / 70 %
        wl = dict(bench.WORKLOADS["qwen3-2layers-bs16-32k-cpu0"], share=(num, 10))
        bench.WORKLOADS["_tmp"] = wl
        try:
            _run_step_and_check("_tmp", [(1, num)])
        finally:
            del bench.WORKLOADS["_tmp"]


def test_qwen3_32k_streamed_load_reading_sampled():
    """The load reading of the same configuration: half of every sequence's P share is not device-resident and comes
    through the slot ring from pinned host memory while the resident rest is attended."""
    stats = _run_step_and_check("qwen3-2layers-bs16-32k-stream50", [(0, 5), (1, 10)])
    # half of 16 x 32 768 tokens x 2 048 bytes went through the slots for each of the two layers
    assert stats["h2d_bytes"] >= 2 * 16 * 16000 * 2048


def test_deepseek_mla_128k_sampled():
    _run_step_and_check("deepseek-v2-lite-mla-2layers-bs8-128k-cpu40", [(0, 0), (1, 7)])


def test_ragged_1m_token_batch_sampled():
    _run_step_and_check("qwen3-ragged-bs64-1m-2layers-cpu30", [(0, 0), (0, 63), (1, 31), (1, 17)])


def test_ragged_1m_token_batch_fixed_schedule_sampled():
    """The same batch at a CPU share of 60 %: short enough for the library to keep the fixed schedule (with the early
    copy start), where the 30 % case above is balanced."""
    wl = dict(bench.WORKLOADS["qwen3-ragged-bs64-1m-2layers-cpu30"], share=(6, 10))
    bench.WORKLOADS["_ragged60"] = wl
    try:
        _run_step_and_check("_ragged60", [(0, 7), (1, 40), (1, 63)])
    finally:
        del bench.WORKLOADS["_ragged60"]


@pytest.mark.parametrize("num,den", [(0, 1), (9, 10)])
def test_ragged_1m_token_batch_at_the_ends_of_the_share_sweep(num, den):
    """CPU share 0 (the longest launches, dynamically balanced, every sequence's ring at its own size) and 90 % (the
    shortest, fixed schedule): the two ends of the sweep, where the planner behaves most differently."""
    wl = dict(bench.WORKLOADS["qwen3-ragged-bs64-1m-2layers-cpu30"], share=(num, den))
    name = f"_ragged_{num}_{den}"
    bench.WORKLOADS[name] = wl
    try:
        _run_step_and_check(name, [(0, 0), (0, 41), (1, 63), (1, 5)])
    finally:
        del bench.WORKLOADS[name]


def _with_workload(name, wl, samples):
    bench.WORKLOADS[name] = wl
    try:
        _run_step_and_check(name, samples)
    finally:
        del bench.WORKLOADS[name]


def test_half_million_token_single_sequence_mla():
    """One very long sequence: 524 288 tokens of compressed-latent cache, every tile of it on one row (the planner cuts
    it into 148 equal chunks); all 16 heads against the oracle."""
    sh = synth.Shape("mla-1l", "mla", 1, 16, 1, 576, 512, 192 ** -0.5)
    _with_workload("_long", dict(shape=sh, batch=1, ctx=1 << 19, share=(0, 1), cfg_id=7), [(0, 0)])


def test_many_short_rows_gqa():
    """256 sequences of 2 048 tokens: more rows than CTA slots in one launch, spans that cross rows inside a CTA."""
    sh = synth.Shape("q-1l", "gqa", 1, 32, 4, 128, 128, 128 ** -0.5)
    _with_workload("_rows", dict(shape=sh, batch=256, ctx=2048, share=(1, 4), cfg_id=8), [(0, 0), (0, 101), (0, 255)])


def test_head_dim_64_and_wide_groups_in_a_cache():
    """head_dim 64 with 24 query heads per KV head (two head groups per KV head) through the handle-based path."""
    sh = synth.Shape("d64", "gqa", 2, 48, 2, 64, 64, 64 ** -0.5)
    _with_workload("_d64", dict(shape=sh, batch=3, ctx=5000, share=(2, 5), cfg_id=9), [(0, 1), (1, 2)])
