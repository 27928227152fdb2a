"""Test-side restatement of the documented block layouts (include/ipkv.h), written from the header text:
used to check region contents byte for byte.  bf16 data as NumPy uint16."""
import numpy as np


def tile_plane(rows_u16, bt):
    """rows_u16 [bt][d] -> flat uint16 plane in TILE layout: d/64 panels of bt rows x 64 columns, the
    8-column (16-byte) chunk c of row t stored at chunk position c ^ (t & 7)."""
    d = rows_u16.shape[1]
    out = np.zeros(bt * d, dtype=np.uint16)
    for t in range(rows_u16.shape[0]):
        for c in range(d // 8):
            panel, cc = divmod(c, 8)
            pos = panel * bt * 64 + t * 64 + ((cc ^ (t & 7)) * 8)
            out[pos:pos + 8] = rows_u16[t, c * 8:(c + 1) * 8]
    return out


def block_image(k, v, bt, layout_tile):
    """k [n][Hkv][dqk], v [n][Hkv][dv] or None, n <= bt -> the block's uint16 image (unwritten rows zero)."""
    n, hkv, dqk = k.shape
    parts = []
    for g in range(hkv):
        kp = np.zeros((bt, dqk), dtype=np.uint16)
        kp[:n] = k[:, g]
        parts.append(tile_plane(kp, bt) if layout_tile else kp.reshape(-1))
        if v is not None:
            vp = np.zeros((bt, v.shape[2]), dtype=np.uint16)
            vp[:n] = v[:, g]
            parts.append(tile_plane(vp, bt) if layout_tile else vp.reshape(-1))
    return np.concatenate(parts)


def blocks_image(k, v, bt, layout_tile):
    """Consecutive blocks holding tokens 0..n-1."""
    n = k.shape[0]
    out = []
    for b in range(0, n, bt):
        out.append(block_image(k[b:b + bt], None if v is None else v[b:b + bt], bt, layout_tile))
    return np.concatenate(out) if out else np.zeros(0, dtype=np.uint16)
