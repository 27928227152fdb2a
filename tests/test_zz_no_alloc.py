"""The allocation-free attention entry point against the ordinary one and against the oracle.

ipkv_attend_runs_noalloc is for callers that cannot allocate device memory where they call attention (a server
whose pool owns all memory, a latency-critical loop, a plug-in that may not allocate): its scratch is a fixed
array inside the library. This file is collected last, so a run that stops at the first failure has already
run every other test. It must pass on its own in a fresh process and after the rest of the suite.
"""
import numpy as np
import pytest

from paper_2609_14507_b200 import binding, synth
from tests.gpu_util import check_partial, oracle_rows, pack_run, shape_of

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _case(seed, rows, hq=32, hkv=4, d=128, bt=64):
    shape = shape_of(binding.GQA, hq, hkv, d, d, bt)
    rng = np.random.default_rng(seed)
    q = synth.bits_to_torch(synth.normal_bf16(rng, (len(rows), hq, d)), "cuda:0")
    bufs, runs = [], []
    for row in rows:
        rr = []
        for n in row:
            buf = pack_run(shape, synth.normal_bf16(rng, (n, hkv, d)), synth.normal_bf16(rng, (n, hkv, d)))
            bufs.append(buf); rr.append((buf, n))
        runs.append(rr)
    return shape, q, runs, bufs


def _both(shape, q, runs, kv_splits):
    n_rows = len(runs)
    total = sum(n for row in runs for _, n in row)
    n_runs = sum(len(row) for row in runs)
    scratch = torch.zeros(binding.ipkv_attend_scratch_bytes(shape, n_rows, n_runs, total, kv_splits), dtype=torch.uint8, device="cuda:0")
    outs = []
    for use_static in (False, True):
        o = torch.full((n_rows, shape.n_q_heads, shape.dim_v), float("nan"), device="cuda:0")
        lse = torch.full((n_rows, shape.n_q_heads), float("nan"), device="cuda:0")
        status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
        if use_static:
            binding.ipkv_attend_runs_noalloc(shape, runs, q, o, lse, kv_splits, status)
        else:
            binding.ipkv_attend_runs(shape, runs, q, scratch, o, lse, kv_splits, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        outs.append((o.cpu().numpy(), lse.cpu().numpy()))
    return outs


def test_noalloc_matches_scratch_variant_on_two_calls_in_a_row():
    # Two different problems back to back: the second call finds the first call's tables and partials in the
    # shared array and must not be affected by them.
    for seed, rows, splits in [(71, [[3000, 130], [64], []], 0), (72, [[900], [2500, 1], [77]], 4)]:
        shape, q, runs, _keep = _case(seed, rows)
        (o_ref, l_ref), (o, l) = _both(shape, q, runs, splits)
        assert np.array_equal(np.isneginf(l), np.isneginf(l_ref))
        fin = np.isfinite(l_ref)
        np.testing.assert_allclose(o, o_ref, atol=2e-3, rtol=0)
        np.testing.assert_allclose(l[fin], l_ref[fin], atol=1e-3, rtol=0)
        # same kernels, same plan: in fact identical
        np.testing.assert_array_equal(o, o_ref)


def test_noalloc_rejects_problems_beyond_its_array():
    shape = shape_of(binding.GQA, 32, 4, 128, 128, 64)
    limit = binding.ipkv_noalloc_scratch_limit()
    assert limit == 16 << 20
    # many splits of a large batch need more partial storage than the array holds; nothing is launched
    rows = [[(1 << 20, 70000)] for _ in range(64)]            # pointers are never dereferenced: the call is refused first
    assert binding.ipkv_attend_scratch_bytes(shape, 64, 64, 64 * 70000, 64) > limit
    q = torch.zeros((64, 32, 128), dtype=torch.bfloat16, device="cuda:0")
    o = torch.zeros((64, 32, 128), device="cuda:0"); lse = torch.zeros((64, 32), device="cuda:0")
    with pytest.raises(binding.IpkvError) as e:
        binding.ipkv_attend_runs_noalloc(shape, rows, q, o, lse, kv_splits=64)
    assert e.value.status == 3
    torch.cuda.synchronize()


@pytest.mark.parametrize("kind", ["gqa", "mla"])
def test_noalloc_matches_the_oracle(kind):
    """The call judged on its own, not through the ordinary entry point: element-wise against the float64 oracle."""
    rng = np.random.default_rng(81)
    rows = [[1500, 70], [333], []]
    if kind == "gqa":
        hq, hkv, dqk, dv, scale = 32, 4, 128, 128, 128 ** -0.5
        shape = shape_of(binding.GQA, hq, hkv, dqk, dv, 64)
    else:
        hq, hkv, dqk, dv, scale = 16, 1, 576, 512, 192 ** -0.5
        shape = shape_of(binding.MLA, hq, hkv, dqk, dv, 64, scale)
    q = synth.normal_bf16(rng, (len(rows), hq, dqk))
    keep, runs, rows_kv = [], [], []
    for row in rows:
        ks, vs, rr = [], [], []
        for n in row:
            k = synth.normal_bf16(rng, (n, hkv, dqk))
            v = None if kind == "mla" else synth.normal_bf16(rng, (n, hkv, dv))
            buf = pack_run(shape, k, v)
            keep.append(buf); rr.append((buf, n)); ks.append(k); vs.append(v)
        runs.append(rr)
        kk = np.concatenate(ks) if ks else np.zeros((0, hkv, dqk), np.uint16)
        vv = None if kind == "mla" else (np.concatenate(vs) if vs else np.zeros((0, hkv, dv), np.uint16))
        rows_kv.append((kk, vv))
    o = torch.full((len(rows), hq, dv), float("nan"), device="cuda:0")
    lse = torch.full((len(rows), hq), float("nan"), device="cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    binding.ipkv_attend_runs_noalloc(shape, runs, synth.bits_to_torch(q, "cuda:0"), o, lse, 3, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    o_ref, l_ref = oracle_rows(q, rows_kv, float(np.float32(scale)), dv_alias=dv if kind == "mla" else None)
    check_partial(o.cpu().numpy(), lse.cpu().numpy(), o_ref, l_ref, f"noalloc {kind}")


def test_noalloc_leaves_device_memory_as_it_found_it():
    """What the name promises: across a hundred calls neither the driver's free memory nor the caller's own allocator
    moves.  The measurement starts after a first burst of the same hundred calls: the first call on a device makes the
    driver set the array aside, and a fresh process's first queue of launches this deep makes the driver grow its own
    launch buffers once; neither is an allocation by the call."""
    shape, q, runs, _keep = _case(82, [[2000, 64], [500]])
    o = torch.zeros((2, shape.n_q_heads, shape.dim_v), device="cuda:0")
    lse = torch.zeros((2, shape.n_q_heads), device="cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")

    def burst():
        for _ in range(100):
            binding.ipkv_attend_runs_noalloc(shape, runs, q, o, lse, 2, status)
        torch.cuda.synchronize()
        return torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved()

    import gc
    gc.collect()                    # tensors of earlier tests must not be released in the middle of the measurement
    burst()
    before = burst()
    after = burst()
    assert after == before, (before, after)
    assert int(status.item()) == 0


def test_noalloc_accepts_the_largest_problem_that_fits_and_refuses_the_next():
    """The limit is the array's 16 MiB: with one 64-token run per row and no explicit splits, the largest batch whose
    scratch still fits is computed (all rows share one run), and one row more is refused with IPKV_ERANGE."""
    shape = shape_of(binding.GQA, 32, 4, 128, 128, 64)
    limit = binding.ipkv_noalloc_scratch_limit()
    need = lambda n: binding.ipkv_attend_scratch_bytes(shape, n, n, 64 * n, 0)
    n = 1
    while need(n + 1) <= limit:
        n += 1
    assert need(n) <= limit < need(n + 1) and n > 64
    rng = np.random.default_rng(83)
    k = synth.normal_bf16(rng, (64, 4, 128)); v = synth.normal_bf16(rng, (64, 4, 128))
    buf = pack_run(shape, k, v)
    q = synth.normal_bf16(rng, (n + 1, 32, 128))
    qd = synth.bits_to_torch(q, "cuda:0")
    o = torch.full((n + 1, 32, 128), float("nan"), device="cuda:0"); lse = torch.full((n + 1, 32), float("nan"), device="cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    binding.ipkv_attend_runs_noalloc(shape, [[(buf, 64)]] * n, qd[:n], o[:n], lse[:n], 0, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    sample = [0, n // 2, n - 1]
    o_ref, l_ref = oracle_rows(q[sample], [(k, v)] * len(sample), float(np.float32(128 ** -0.5)))
    check_partial(o.cpu().numpy()[sample], lse.cpu().numpy()[sample], o_ref, l_ref, "noalloc at the limit")
    assert torch.isfinite(o[:n]).all()
    with pytest.raises(binding.IpkvError) as e:
        binding.ipkv_attend_runs_noalloc(shape, [[(buf, 64)]] * (n + 1), qd, o, lse, 0, status)
    assert e.value.status == 3                                     # IPKV_ERANGE, nothing launched
    torch.cuda.synchronize()


@pytest.mark.parametrize("kind", ["gqa", "mla"])
def test_stateless_call_can_be_recorded_into_a_cuda_graph(kind):
    """Under stream capture the launch tables travel as kernel parameters (a captured copy from the call's temporary
    host image would be replayed after the image is gone), so the recorded graph can be replayed: it gives the bits of
    a direct call, and follows new queries written into the same buffer."""
    if kind == "gqa":
        shape, q, runs, _keep = _case(73, [[1500, 64], [700], [33]])
    else:
        shape = shape_of(binding.MLA, 16, 1, 576, 512, 64)
        rng = np.random.default_rng(74)
        q = synth.bits_to_torch(synth.normal_bf16(rng, (2, 16, 576)), "cuda:0")
        _keep = [pack_run(shape, synth.normal_bf16(rng, (n, 1, 576)), None) for n in (900, 130)]
        runs = [[(_keep[0], 900)], [(_keep[1], 130)]]
    n_rows = len(runs)

    def direct():
        o = torch.full((n_rows, shape.n_q_heads, shape.dim_v), float("nan"), device="cuda:0")
        lse = torch.full((n_rows, shape.n_q_heads), float("nan"), device="cuda:0")
        binding.ipkv_attend_runs_noalloc(shape, runs, q, o, lse, 2)
        torch.cuda.synchronize()
        return o.clone(), lse.clone()

    o_ref, l_ref = direct()                                  # also resolves the array's address outside the capture
    o_g = torch.full((n_rows, shape.n_q_heads, shape.dim_v), float("nan"), device="cuda:0")
    l_g = torch.full((n_rows, shape.n_q_heads), float("nan"), device="cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        binding.ipkv_attend_runs_noalloc(shape, runs, q, o_g, l_g, 2, status)
    torch.cuda.synchronize()
    assert torch.isnan(o_g).all()                            # recording ran nothing
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(o_g, o_ref) and torch.equal(l_g, l_ref) and int(status.item()) == 0
    q.copy_(synth.bits_to_torch(synth.normal_bf16(np.random.default_rng(75), tuple(q.shape)), "cuda:0"))
    o_ref2, l_ref2 = direct()
    assert not torch.equal(o_ref2, o_ref)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(o_g, o_ref2) and torch.equal(l_g, l_ref2)
