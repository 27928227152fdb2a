"""GPU parity of the stateless kernel entry points against the float64 oracle, through the C ABI."""
import numpy as np
import pytest

from oracle import c_oracle
from paper_2609_14507_b200 import binding, synth
from tests import layouts
from tests.gpu_util import check_partial, oracle_rows, pack_run, shape_of

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.mark.parametrize("kind,hkv,dqk,dv", [(binding.GQA, 4, 128, 128), (binding.GQA, 2, 64, 64), (binding.MLA, 1, 576, 512)])
@pytest.mark.parametrize("bt", [16, 64, 128])
@pytest.mark.parametrize("layout", [binding.LAYOUT_PLAIN, binding.LAYOUT_TILE])
def test_pack_blocks_is_bit_exact(kind, hkv, dqk, dv, bt, layout):
    shape = shape_of(kind, 16 * hkv if kind == binding.GQA else 16, hkv, dqk, dv, bt)
    rng = np.random.default_rng(41)
    n = 3 * bt + 5
    k = synth.normal_bf16(rng, (n, hkv, dqk))
    v = None if kind == binding.MLA else synth.normal_bf16(rng, (n, hkv, dv))
    buf = pack_run(shape, k, v, layout)
    got = buf.cpu().numpy().view(np.uint16)
    want = layouts.blocks_image(k, v, bt, layout == binding.LAYOUT_TILE)
    np.testing.assert_array_equal(got, want)


GQA_CASES = [
    # (Hq, Hkv, d, bt, run lengths per row, kv_splits)
    (32, 4, 128, 64, [[4096 + 1]], 0),
    (32, 4, 128, 64, [[1]], 0),
    (32, 8, 128, 64, [[700, 33], [64], [1000, 1, 129]], 0),
    (32, 4, 128, 64, [[2049], [], [517, 255]], 3),
    (32, 4, 128, 64, [[2049], [300]], 1),
    (8, 8, 128, 64, [[333]], 0),                  # MHA: groups of one head
    (16, 1, 128, 64, [[450, 70]], 0),             # MQA: all 16 heads share the KV head
    (40, 1, 128, 64, [[450]], 0),                 # more than 16 heads per KV head: several head groups
    (12, 4, 64, 64, [[1500, 77]], 0),             # head_dim 64, odd group size 3
    (32, 4, 128, 16, [[1000, 17], [15]], 0),      # small blocks: tiles span several blocks
    (32, 4, 128, 32, [[1000, 33]], 2),
    (32, 4, 128, 128, [[1000, 257]], 0),          # large blocks: several tiles per block
    (32, 4, 128, 256, [[5000, 100], [256]], 0),
    (32, 4, 128, 64, [[6400], [6208]], 4),        # ragged rows with explicit splits: CTA cuts fall inside the pieces
]


@pytest.mark.parametrize("hq,hkv,d,bt,rows,kv_splits", GQA_CASES)
def test_attend_runs_gqa_matches_oracle(hq, hkv, d, bt, rows, kv_splits):
    shape = shape_of(binding.GQA, hq, hkv, d, d, bt)
    scale = d ** -0.5
    rng = np.random.default_rng(42)
    n_rows = len(rows)
    q = synth.normal_bf16(rng, (n_rows, hq, d))
    bufs, runs, rows_kv = [], [], []
    for row in rows:
        ks, vs, rr = [], [], []
        for n in row:
            k = synth.normal_bf16(rng, (n, hkv, d)); v = synth.normal_bf16(rng, (n, hkv, d))
            buf = pack_run(shape, k, v)
            bufs.append(buf); rr.append((buf, n)); ks.append(k); vs.append(v)
        runs.append(rr)
        rows_kv.append((np.concatenate(ks) if ks else np.zeros((0, hkv, d), np.uint16),
                        np.concatenate(vs) if vs else np.zeros((0, hkv, d), np.uint16)))
    total = sum(sum(r) for r in rows)
    n_runs = sum(len(r) for r in rows)
    scratch = torch.zeros(binding.ipkv_attend_scratch_bytes(shape, n_rows, n_runs, total, kv_splits), dtype=torch.uint8, device="cuda:0")
    o = torch.full((n_rows, hq, d), float("nan"), device="cuda:0")
    lse = torch.full((n_rows, hq), float("nan"), device="cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    binding.ipkv_attend_runs(shape, runs, synth.bits_to_torch(q, "cuda:0"), scratch, o, lse, kv_splits, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    o_ref, lse_ref = oracle_rows(q, rows_kv, float(np.float32(scale)))
    check_partial(o.cpu().numpy(), lse.cpu().numpy(), o_ref, lse_ref, f"{hq}/{hkv} d{d} bt{bt}")


def test_attend_runs_peaked_softmax_and_identical_keys():
    # O of order one, so the absolute tolerance binds: identical keys give the mean of V; one dominant key gives its V.
    hq, hkv, d, bt, n = 32, 4, 128, 64, 777
    shape = shape_of(binding.GQA, hq, hkv, d, d, bt)
    rng = np.random.default_rng(43)
    q = synth.normal_bf16(rng, (2, hq, d))
    k_same = np.repeat(synth.normal_bf16(rng, (1, hkv, d)), n, axis=0)
    v0 = synth.normal_bf16(rng, (n, hkv, d))
    k_dom = synth.f32_to_bf16_bits(rng.standard_normal((n, hkv, d)).astype(np.float32) * 0.05)
    qf = synth.bf16_bits_to_f32(q[1]).reshape(hkv, hq // hkv, d)
    k_dom[555] = synth.f32_to_bf16_bits(8.0 * np.sign(qf.sum(axis=1)))          # aligned with the group's queries
    v1 = synth.normal_bf16(rng, (n, hkv, d))
    b0, b1 = pack_run(shape, k_same, v0), pack_run(shape, k_dom, v1)
    scratch = torch.zeros(binding.ipkv_attend_scratch_bytes(shape, 2, 2, 2 * n, 0), dtype=torch.uint8, device="cuda:0")
    o = torch.zeros((2, hq, d), device="cuda:0"); lse = torch.zeros((2, hq), device="cuda:0")
    binding.ipkv_attend_runs(shape, [[(b0, n)], [(b1, n)]], synth.bits_to_torch(q, "cuda:0"), scratch, o, lse)
    torch.cuda.synchronize()
    o_ref, lse_ref = oracle_rows(q, [(k_same, v0), (k_dom, v1)], float(np.float32(d ** -0.5)))
    check_partial(o.cpu().numpy(), lse.cpu().numpy(), o_ref, lse_ref, "structured")
    mean_v = synth.bf16_bits_to_f32(v0).astype(np.float64).mean(axis=0)          # [hkv][d]
    np.testing.assert_allclose(o[0].cpu().numpy().reshape(hkv, hq // hkv, d), np.repeat(mean_v[:, None], hq // hkv, 1), atol=2e-3)


@pytest.mark.parametrize("n_parts,dv,bf16_out", [(2, 128, False), (2, 512, True), (5, 128, False), (8, 64, True), (1, 128, False)])
def test_merge_matches_oracle(n_parts, dv, bf16_out):
    rng = np.random.default_rng(44)
    rows = 37
    Os = rng.standard_normal((n_parts, rows, dv)).astype(np.float32)
    Ls = (rng.standard_normal((n_parts, rows)) * 4).astype(np.float32)
    Ls[0, 3] = -np.inf
    Ls[:, 5] = -np.inf                                   # a row nobody attended
    Os[:, 5] = 0
    o_parts = [torch.from_numpy(Os[i]).cuda() for i in range(n_parts)]
    l_parts = [torch.from_numpy(Ls[i]).cuda() for i in range(n_parts)]
    out = torch.zeros((rows, dv), dtype=torch.bfloat16 if bf16_out else torch.float32, device="cuda:0")
    lse = torch.zeros(rows, device="cuda:0")
    binding.ipkv_merge(rows, dv, o_parts, l_parts, out, lse, out_is_bf16=bf16_out)
    torch.cuda.synchronize()
    o_ref, l_ref = c_oracle.merge([(Os[i].astype(np.float64), Ls[i].astype(np.float64)) for i in range(n_parts)])
    got = out.float().cpu().numpy().astype(np.float64)
    tol = 2 ** -8 if bf16_out else 1e-5
    np.testing.assert_allclose(got, o_ref, rtol=tol, atol=1e-5)
    gl = lse.cpu().numpy().astype(np.float64)
    assert np.array_equal(np.isneginf(gl), np.isneginf(l_ref))
    np.testing.assert_allclose(gl[np.isfinite(l_ref)], l_ref[np.isfinite(l_ref)], atol=1e-5, rtol=1e-6)


MLA_CASES = [
    # (Hq, bt, run lengths per row, kv_splits)
    (16, 64, [[4096 + 1]], 0),
    (16, 64, [[700, 33], [64], [1]], 0),
    (16, 64, [[2049], [], [517, 255]], 3),
    (32, 64, [[500]], 0),                    # two groups of 16 heads
    (5, 64, [[300, 10]], 0),                 # fewer than 16 heads
    (16, 16, [[1000, 17]], 0),
    (16, 32, [[70]], 0),
    (16, 128, [[1000, 257]], 2),
    (16, 64, [[6400], [6208]], 8),           # ragged rows with explicit splits: CTA cuts fall inside the pieces
]


@pytest.mark.parametrize("hq,bt,rows,kv_splits", MLA_CASES)
def test_attend_runs_mla_matches_oracle(hq, bt, rows, kv_splits):
    """Compressed-latent kind: cached row = [latent 512 | rope 64], V = the row's first 512 columns."""
    scale = 192 ** -0.5
    shape = shape_of(binding.MLA, hq, 1, 576, 512, bt, scale)
    rng = np.random.default_rng(45)
    n_rows = len(rows)
    q = synth.normal_bf16(rng, (n_rows, hq, 576))
    bufs, runs, rows_kv = [], [], []
    for row in rows:
        ks, rr = [], []
        for n in row:
            k = synth.normal_bf16(rng, (n, 1, 576))
            buf = pack_run(shape, k, None)
            bufs.append(buf); rr.append((buf, n)); ks.append(k)
        runs.append(rr)
        rows_kv.append((np.concatenate(ks) if ks else np.zeros((0, 1, 576), np.uint16), None))
    total = sum(sum(r) for r in rows)
    n_runs = sum(len(r) for r in rows)
    scratch = torch.zeros(binding.ipkv_attend_scratch_bytes(shape, n_rows, n_runs, total, kv_splits), dtype=torch.uint8, device="cuda:0")
    o = torch.full((n_rows, hq, 512), float("nan"), device="cuda:0")
    lse = torch.full((n_rows, hq), float("nan"), device="cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    binding.ipkv_attend_runs(shape, runs, synth.bits_to_torch(q, "cuda:0"), scratch, o, lse, kv_splits, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    o_ref, lse_ref = oracle_rows(q, rows_kv, float(np.float32(scale)), dv_alias=512)
    check_partial(o.cpu().numpy(), lse.cpu().numpy(), o_ref, lse_ref, f"mla {hq} heads bt{bt}")


def test_attend_runs_mla_peaked_softmax():
    hq, bt, n = 16, 64, 333
    scale = 192 ** -0.5
    shape = shape_of(binding.MLA, hq, 1, 576, 512, bt, scale)
    rng = np.random.default_rng(46)
    q = synth.normal_bf16(rng, (1, hq, 576))
    k = synth.f32_to_bf16_bits(rng.standard_normal((n, 1, 576)).astype(np.float32) * 0.05)
    qf = synth.bf16_bits_to_f32(q[0])
    k[100, 0] = synth.f32_to_bf16_bits(3.0 * np.sign(qf.sum(axis=0)))
    k[7, 0] = synth.f32_to_bf16_bits(rng.standard_normal(576).astype(np.float32))
    buf = pack_run(shape, k, None)
    scratch = torch.zeros(binding.ipkv_attend_scratch_bytes(shape, 1, 1, n, 0), dtype=torch.uint8, device="cuda:0")
    o = torch.zeros((1, hq, 512), device="cuda:0"); lse = torch.zeros((1, hq), device="cuda:0")
    binding.ipkv_attend_runs(shape, [[(buf, n)]], synth.bits_to_torch(q, "cuda:0"), scratch, o, lse)
    torch.cuda.synchronize()
    o_ref, lse_ref = oracle_rows(q, [(k, None)], float(np.float32(scale)), dv_alias=512)
    assert np.abs(o_ref).max() > 0.5                       # O of order one: the absolute tolerance binds
    check_partial(o.cpu().numpy(), lse.cpu().numpy(), o_ref, lse_ref, "mla peaked")


def test_mla_tcgen05_variant_matches_oracle():
    """The opt-in tcgen05 / TMEM kernel (IPKV_MLA_TC=1) passes the same MLA parity cases; run in a child process
    because the switch is read once per process."""
    import os
    import subprocess
    import sys
    env = dict(os.environ, IPKV_MLA_TC="1")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-m", "gpu", "-x", os.path.join(root, "tests", "test_gpu_kernels.py"),
                        "-k", "attend_runs_mla"], env=env, cwd=root, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]


def test_bounds_checked_build_passes_the_small_parity_cases():
    """The -DIPKV_CHECKED build of the same kernels (every computed source address, partial row and window slot compared
    with its region's extent; the stand-in for a memory checker) runs the small-shape parity tests of both attention
    kernels, the handle-based decode tests and its own self-test without recording a violation where none is planted.
    A child process, because the library variant is chosen when the library is first loaded."""
    import os
    import subprocess
    import sys
    env = dict(os.environ, IPKV_LIB_VARIANT="checked")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-m", "gpu", "-x", os.path.join(root, "tests", "test_gpu_kernels.py"),
                        os.path.join(root, "tests", "test_gpu_cache.py"), "-k",
                        "attend_runs_gqa or attend_runs_mla or peaked or config1 or decode_steps or ring_capacity or fused or checked_build_records"],
                       env=env, cwd=root, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "skipped" not in r.stdout.splitlines()[-1]


@pytest.mark.parametrize("parts,variant", [("1", ""), ("4", ""), ("1", "checked")])
def test_both_forms_of_the_span_partial_pass_the_small_parity_cases(parts, variant):
    """The grouped-query kernel writes one partial per span (its four warps join their states through shared memory) in
    launches with long spans and four otherwise; small cases would only ever see the second form.  Here each form is
    forced in turn (IPKV_PARTS_PER_SPAN, read when the library is first used: a child process) and the small-shape parity
    tests, ragged and balanced cases and the decode tests run against it; the joined form also in the bounds-checked build."""
    import os
    import subprocess
    import sys
    env = dict(os.environ, IPKV_PARTS_PER_SPAN=parts)
    if variant:
        env["IPKV_LIB_VARIANT"] = variant
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-m", "gpu", "-x", os.path.join(root, "tests", "test_gpu_kernels.py"),
                        os.path.join(root, "tests", "test_gpu_cache.py"), "-k",
                        "attend_runs_gqa or peaked or identical or config1 or decode_steps or fused or static_schedule or balanc or sparse"],
                       env=env, cwd=root, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout


def test_read_bandwidth_probe_runs():
    """The measurement aid behind `roofline.read_ceiling`: a read-only stream through the kernels' copy ring."""
    best, mean = binding.ipkv_probe_read_bandwidth(0, 256 << 20, 3)
    assert 500.0 < mean <= best < 20000.0
    with pytest.raises(binding.IpkvError):
        binding.ipkv_probe_read_bandwidth(0, 1 << 20, 3)          # below the 64 MB minimum
