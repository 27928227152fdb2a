"""Helpers shared by the GPU parity tests: tolerances, oracle calls on the same bits, block builders."""
import numpy as np

from oracle import c_oracle
from paper_2609_14507_b200 import binding, synth

# Tolerances for bf16 inputs with fp32 accumulation (the probabilities are rounded to bf16 before the
# P.V product; everything else is fp32): O max-abs 2e-3 and row-normalised max-rel 1e-2, LSE abs 1e-3.
O_ATOL, O_ROW_RTOL, LSE_ATOL = 2e-3, 1e-2, 1e-3


def check_partial(o, lse, o_ref, lse_ref, what=""):
    o = np.asarray(o, dtype=np.float64); lse = np.asarray(lse, dtype=np.float64)
    assert o.shape == o_ref.shape and lse.shape == lse_ref.shape, (o.shape, o_ref.shape)
    assert np.all(np.isfinite(o)), what
    inf_ref = np.isneginf(lse_ref)
    assert np.array_equal(np.isneginf(lse), inf_ref), what
    if inf_ref.any():
        assert np.all(o[inf_ref] == 0.0), what
    fin = ~inf_ref
    err = np.abs(o - o_ref)
    assert err.max(initial=0.0) <= O_ATOL, f"{what}: O max-abs {err.max():.3e}"
    if fin.any():
        row_scale = np.abs(o_ref[fin]).max(axis=-1)
        row_err = err[fin].max(axis=-1)
        rel = row_err / np.maximum(row_scale, 1e-30)
        assert rel.max() <= O_ROW_RTOL, f"{what}: O row-normalised max-rel {rel.max():.3e}"
        lerr = np.abs(lse[fin] - lse_ref[fin]).max()
        assert lerr <= LSE_ATOL, f"{what}: LSE abs {lerr:.3e}"


def shape_of(kind, hq, hkv, dqk, dv, bt, scale=0.0):
    return binding.make_shape(kind, hq, hkv, dqk, dv, bt, scale)


def pack_run(shape, k_bits, v_bits, layout=binding.LAYOUT_TILE, device="cuda:0"):
    """Host bf16 bits -> a device buffer of consecutive blocks in the given layout (zero padded)."""
    import torch
    n = k_bits.shape[0]
    bb = binding.ipkv_block_bytes(shape)
    nb = max(1, -(-n // shape.block_tokens))
    buf = torch.zeros(nb * bb, dtype=torch.uint8, device=device)
    kd = synth.bits_to_torch(k_bits, device)
    vd = synth.bits_to_torch(v_bits, device) if v_bits is not None else None
    binding.ipkv_pack_blocks(shape, layout, kd, vd, n, buf)
    return buf


def oracle_rows(q_bits, rows_kv, scale, dv_alias=None):
    """q_bits [rows][Hq][dqk]; rows_kv[r] = (K [n][Hkv][dqk], V or None). -> (O [rows][Hq][dv], LSE [rows][Hq])."""
    Os, Ls = [], []
    for r, (k, v) in enumerate(rows_kv):
        vv = dv_alias if v is None else v
        o, l = c_oracle.attend(q_bits[r], k, vv, np.arange(k.shape[0]), scale)
        Os.append(o); Ls.append(l)
    return np.stack(Os), np.stack(Ls)
