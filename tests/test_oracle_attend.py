"""Pins for the attention oracle (O1): closed forms, invariants, library special cases.

Each pin is chosen so that a plausible slip in the oracle (wrong head mapping, dropped scale,
transposed operand, log base, missing normalisation) fails at least one of them.
"""
import math

import numpy as np
import pytest

from oracle import c_oracle, np_oracle
from paper_2609_14507_b200 import synth

IMPLS = [pytest.param(c_oracle.attend, id="cpp"), pytest.param(np_oracle.attend, id="numpy")]


def bits(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def f64(b):
    return np_oracle.bf16_bits_to_f64(b)


@pytest.mark.parametrize("attend", IMPLS)
def test_two_tokens_hand_derived(attend):
    # q = e0; k0 = 0 (score 0), k1 = (ln 3 / scale) e0 is not bf16-exact, so use exact values instead:
    # scale = 1, q = (1, 0), k0 = (0, 0), k1 = (2, 0): scores 0 and 2 -> weights 1/(1+e^2), e^2/(1+e^2).
    q = bits([[1.0, 0.0]])
    k = bits([[[0.0, 0.0]], [[2.0, 0.0]]])
    v = bits([[[1.0, -1.0]], [[3.0, 5.0]]])
    O, lse = attend(q, k, v, [0, 1], 1.0)
    w1 = math.exp(2.0) / (1.0 + math.exp(2.0))
    np.testing.assert_allclose(O[0], [(1 - w1) * 1 + w1 * 3, (1 - w1) * -1 + w1 * 5], rtol=1e-14)
    assert lse[0] == pytest.approx(math.log(1.0 + math.exp(2.0)), rel=1e-15)


@pytest.mark.parametrize("attend", IMPLS)
def test_scale_enters_scores_and_lse(attend):
    # scores scale*4 and 0 with scale = 0.25 -> 1 and 0: LSE = ln(1 + e)
    q = bits([[2.0, 0.0]])
    k = bits([[[2.0, 7.0]], [[0.0, -3.0]]])
    v = bits([[[8.0]], [[-8.0]]])
    O, lse = attend(q, k, v, [0, 1], 0.25)
    assert lse[0] == pytest.approx(math.log(1.0 + math.e), rel=1e-15)
    assert O[0, 0] == pytest.approx(8.0 * (math.e - 1.0) / (math.e + 1.0), rel=1e-14)


@pytest.mark.parametrize("attend", IMPLS)
def test_single_token_returns_its_value(attend):
    rng = np.random.default_rng(1)
    q = synth.normal_bf16(rng, (8, 16))
    k = synth.normal_bf16(rng, (5, 2, 16))
    v = synth.normal_bf16(rng, (5, 2, 24))
    O, lse = attend(q, k, v, [3], 0.3)
    for h in range(8):
        g = h // 4
        np.testing.assert_array_equal(O[h], f64(v[3, g]))
        assert lse[h] == pytest.approx(0.3 * float(f64(q[h]) @ f64(k[3, g])), rel=1e-14)


@pytest.mark.parametrize("attend", IMPLS)
def test_identical_keys_give_mean_of_values(attend):
    rng = np.random.default_rng(2)
    N, Hq, Hkv, d = 37, 8, 2, 32
    q = synth.normal_bf16(rng, (Hq, d))
    k1 = synth.normal_bf16(rng, (1, Hkv, d))
    k = np.repeat(k1, N, axis=0)
    v = synth.normal_bf16(rng, (N, Hkv, d))
    O, lse = attend(q, k, v, np.arange(N), 0.17)
    for h in range(Hq):
        g = h // (Hq // Hkv)
        np.testing.assert_allclose(O[h], f64(v[:, g]).mean(axis=0), rtol=1e-13, atol=1e-15)
        s = 0.17 * float(f64(q[h]) @ f64(k1[0, g]))
        assert lse[h] == pytest.approx(s + math.log(N), rel=1e-13)


@pytest.mark.parametrize("attend", IMPLS)
def test_dominant_key_selects_its_value(attend):
    rng = np.random.default_rng(3)
    N, d = 50, 16
    q = bits(np.full((1, d), 4.0))
    kf = rng.standard_normal((N, 1, d)).astype(np.float32) * 0.01
    kf[17, 0, :] = 4.0                       # score gap ~ 16*d*scale = 256 with scale 1
    v = synth.normal_bf16(rng, (N, 1, d))
    O, lse = attend(q, bits(kf), v, np.arange(N), 1.0)
    np.testing.assert_allclose(O[0], f64(v[17, 0]), rtol=0, atol=1e-60)
    assert lse[0] == pytest.approx(16.0 * d, rel=1e-15)


@pytest.mark.parametrize("attend", IMPLS)
def test_permutation_and_subset_semantics(attend):
    rng = np.random.default_rng(4)
    q = synth.normal_bf16(rng, (4, 32))
    k = synth.normal_bf16(rng, (64, 2, 32))
    v = synth.normal_bf16(rng, (64, 2, 32))
    idx = rng.choice(64, size=40, replace=False)
    O1, l1 = attend(q, k, v, idx, 0.2)
    O2, l2 = attend(q, k, v, rng.permutation(idx), 0.2)
    np.testing.assert_allclose(O1, O2, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(l1, l2, rtol=1e-13)
    # only the listed tokens matter: compact the subset and attend over all of it
    O3, l3 = attend(q, k[np.sort(idx)], v[np.sort(idx)], np.arange(40), 0.2)
    np.testing.assert_allclose(O1, O3, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(l1, l3, rtol=1e-13)


@pytest.mark.parametrize("attend", IMPLS)
def test_empty_set(attend):
    rng = np.random.default_rng(5)
    q = synth.normal_bf16(rng, (4, 8))
    k = synth.normal_bf16(rng, (3, 1, 8))
    v = synth.normal_bf16(rng, (3, 1, 8))
    O, lse = attend(q, k, v, [], 1.0)
    assert np.all(O == 0.0) and np.all(np.isneginf(lse))


@pytest.mark.parametrize("attend", IMPLS)
def test_score_shift_moves_lse_only(attend):
    # Append a constant feature: q gets 1, every key gets c/scale. All scores grow by c exactly
    # (c/scale chosen bf16-exact), so O is unchanged and LSE grows by c.
    rng = np.random.default_rng(6)
    N, d, scale, c = 20, 15, 0.5, 3.0
    qf = rng.standard_normal((2, d)).astype(np.float32)
    kf = rng.standard_normal((N, 1, d)).astype(np.float32)
    v = synth.normal_bf16(rng, (N, 1, 8))
    q0 = bits(np.concatenate([qf, np.zeros((2, 1), np.float32)], axis=1))
    q1 = bits(np.concatenate([qf, np.ones((2, 1), np.float32)], axis=1))
    k1 = bits(np.concatenate([kf, np.full((N, 1, 1), c / scale, np.float32)], axis=2))
    O0, l0 = attend(q0, k1, v, np.arange(N), scale)
    O1, l1 = attend(q1, k1, v, np.arange(N), scale)
    np.testing.assert_allclose(O1, O0, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(l1, l0 + c, rtol=1e-13)


@pytest.mark.parametrize("attend", IMPLS)
@pytest.mark.parametrize("Hq,Hkv", [(8, 8), (8, 2), (8, 1), (32, 4)])
def test_against_torch_sdpa_float64(attend, Hq, Hkv):
    # Library special case: torch CPU float64 scaled_dot_product_attention with the KV heads
    # repeated contiguously (query head h -> KV head h // G); MHA and MQA are the G=1 / Hkv=1 ends.
    import torch
    rng = np.random.default_rng(7)
    N, dqk, dv, scale = 129, 64, 48, 0.11
    q = synth.normal_bf16(rng, (Hq, dqk))
    k = synth.normal_bf16(rng, (N, Hkv, dqk))
    v = synth.normal_bf16(rng, (N, Hkv, dv))
    O, lse = attend(q, k, v, np.arange(N), scale)
    G = Hq // Hkv
    tq = torch.from_numpy(f64(q))[None, :, None, :]                                    # [1][Hq][1][d]
    tk = torch.from_numpy(f64(k)).permute(1, 0, 2).repeat_interleave(G, dim=0)[None]   # [1][Hq][N][d]
    tv = torch.from_numpy(f64(v)).permute(1, 0, 2).repeat_interleave(G, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, scale=scale)[0, :, 0, :].numpy()
    np.testing.assert_allclose(O, ref, rtol=1e-11, atol=1e-14)
    from scipy.special import logsumexp
    s = scale * np.einsum("hd,nhd->hn", f64(q), np.repeat(f64(k), G, axis=1))
    np.testing.assert_allclose(lse, logsumexp(s, axis=1), rtol=1e-13)


@pytest.mark.parametrize("attend", IMPLS)
def test_latent_value_alias_equals_explicit_value(attend):
    # Compressed-latent case: V is the leading dv columns of the shared K row (Sec. 6.1).
    rng = np.random.default_rng(8)
    N, Hq, dqk, dv = 33, 16, 72, 64
    q = synth.normal_bf16(rng, (Hq, dqk))
    k = synth.normal_bf16(rng, (N, 1, dqk))
    Oa, la = attend(q, k, dv, np.arange(N), 0.07)
    Ob, lb = attend(q, k, np.ascontiguousarray(k[:, :, :dv]), np.arange(N), 0.07)
    np.testing.assert_array_equal(Oa, Ob)
    np.testing.assert_array_equal(la, lb)


def test_cpp_and_numpy_agree():
    rng = np.random.default_rng(9)
    for (Hq, Hkv, dqk, dv, N) in [(32, 4, 128, 128, 300), (16, 1, 576, 512, 70)]:
        q = synth.normal_bf16(rng, (Hq, dqk))
        k = synth.normal_bf16(rng, (N, Hkv, dqk))
        v = dv if Hkv == 1 else synth.normal_bf16(rng, (N, Hkv, dv))
        idx = np.arange(N)[::2]
        O1, l1 = c_oracle.attend(q, k, v, idx, dqk ** -0.5)
        O2, l2 = np_oracle.attend(q, k, v, idx, dqk ** -0.5)
        np.testing.assert_allclose(O1, O2, rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(l1, l2, rtol=1e-13)


def test_arithmetic_intensity_pin(golden):
    # Sec. 5.2: per KV token and query head, attention does 2d MACs (q.k and p.v) over the
    # 4d bytes of one bf16 K row and one bf16 V row: 0.5 MAC per byte.
    d = 128
    assert (2 * d) / (2 * 2 * d) == golden["sec5_2.mac_per_byte"]
