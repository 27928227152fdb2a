"""NumPy float64 twin of the C++ oracle (TEST INFRASTRUCTURE).

Written independently of ``ipkv_oracle.cpp`` (vectorised, different evaluation order) so that
the two can be checked against each other as well as against the paper's pins.

* :func:`attend`  — the textbook definition of softmax attention over a token set
  (the method is exact: Sec. 4.3 guarantee (iv), Sec. 5.1).
* :func:`merge`, :func:`merge2` — log-sum-exp join of partials over disjoint sets (Sec. 4.2, 5.1).
* :class:`Route` — write-time routing into the regions (Sec. 4.1, 4.2, 5.3), integers only.
* :func:`kv_bytes_per_token`, :func:`footprint` — region sizes (Tables 1 and 2, Sec. 7.7).
"""
import numpy as np

REGION_U, REGION_P, REGION_W = 0, 1, 2


def bf16_bits_to_f64(bits):
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    bits = np.asarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def attend(q, k, v, idx, scale):
    """q [Hq][dqk], k [n][Hkv][dqk], v [n][Hkv][dv] (uint16 bf16 bits) or an int dv (V = K[..., :dv]).

    Query head h reads KV head h // (Hq // Hkv).  Returns (O [Hq][dv], LSE [Hq]); the LSE is the
    natural log of the sum of exp(scale * q.k).  Empty set -> (0, -inf).
    """
    qd = bf16_bits_to_f64(q)
    kd = bf16_bits_to_f64(k)
    vd = kd[..., :v] if isinstance(v, (int, np.integer)) else bf16_bits_to_f64(v)
    Hq, Hkv = qd.shape[0], kd.shape[1]
    G = Hq // Hkv
    idx = np.asarray(idx, dtype=np.int64)
    dv = vd.shape[2]
    O = np.zeros((Hq, dv))
    lse = np.full((Hq,), -np.inf)
    if idx.size == 0:
        return O, lse
    ks, vs = kd[idx], vd[idx]                       # [T][Hkv][d]
    for h in range(Hq):
        s = float(scale) * (ks[:, h // G, :] @ qd[h])
        m = s.max()
        w = np.exp(s - m)
        lse[h] = m + np.log(w.sum())
        O[h] = (w / w.sum()) @ vs[:, h // G, :]
    return O, lse


def merge2(Oa, la, Ob, lb):
    """Two-way join: LSE = logaddexp(la, lb); O = exp(la-LSE) Oa + exp(lb-LSE) Ob."""
    Oa, Ob = np.asarray(Oa, dtype=np.float64), np.asarray(Ob, dtype=np.float64)
    la, lb = np.asarray(la, dtype=np.float64), np.asarray(lb, dtype=np.float64)
    with np.errstate(invalid="ignore"):
        L = np.logaddexp(la, lb)
        wa = np.where(np.isneginf(la), 0.0, np.exp(la - L))
        wb = np.where(np.isneginf(lb), 0.0, np.exp(lb - L))
    return wa[:, None] * Oa + wb[:, None] * Ob, L


def merge(parts):
    """n-way join in one shot over parts = [(O_i [rows][dv], lse_i [rows]), ...]."""
    Os = np.stack([np.asarray(p[0], dtype=np.float64) for p in parts])      # [n][rows][dv]
    Ls = np.stack([np.asarray(p[1], dtype=np.float64) for p in parts])      # [n][rows]
    m = Ls.max(axis=0)
    safe_m = np.where(np.isneginf(m), 0.0, m)
    e = np.exp(Ls - safe_m)                                                   # -inf -> 0
    z = e.sum(axis=0)
    with np.errstate(divide="ignore"):
        L = np.where(z > 0, safe_m + np.log(np.where(z > 0, z, 1.0)), -np.inf)
    w = np.where(z > 0, e / np.where(z > 0, z, 1.0), 0.0)
    return np.einsum("nr,nrd->rd", w, Os), L


class Route:
    """Routing of one (layer, sequence), kept as a list of placed runs rather than per token.

    ``runs`` holds (region, first_token, n_tokens, first_block); the window is [w0, n).
    The k-th flush goes to U iff floor((acc0 + sum of shares so far) / den) increases, acc0 = den // 2.
    """

    def __init__(self, block, D, num, den):
        assert block > 0 and D > 0 and D % block == 0 and den > 0 and 0 <= num <= den
        self.block, self.D, self.num, self.den = block, D, num, den
        self.acc = den // 2
        self.runs = []
        self.next_block = {REGION_U: 0, REGION_P: 0}
        self.n = 0
        self.w0 = 0
        self.n_flush = 0
        self.n_flush_cpu = 0

    def _place(self, region, first, count):
        if count == 0:
            return
        self.runs.append((region, first, count, self.next_block[region]))
        self.next_block[region] += -(-count // self.block)

    def set_share(self, num):
        assert 0 <= num <= self.den
        self.num = num

    def bulk(self, n0, num0, den0):
        assert self.n == 0 and n0 >= 0 and den0 > 0 and 0 <= num0 <= den0
        n_cpu = self.block * ((n0 // self.block) * num0 // den0)
        self._place(REGION_U, 0, n_cpu)
        self._place(REGION_P, n_cpu, n0 - n_cpu)
        self.n = self.w0 = n0

    def flush(self):
        cnt = self.n - self.w0
        if cnt == 0:
            return
        self.acc += self.num
        to_cpu = self.acc >= self.den
        if to_cpu:
            self.acc -= self.den
        self._place(REGION_U if to_cpu else REGION_P, self.w0, cnt)
        self.w0 = self.n
        self.n_flush += 1
        self.n_flush_cpu += int(to_cpu)

    def append(self):
        if self.n - self.w0 == self.D:
            self.flush()
        self.n += 1

    def __len__(self):
        return self.n

    def dump(self):
        region = np.full(self.n, REGION_W, dtype=np.int8)
        blk = np.zeros(self.n, dtype=np.int64)
        off = np.zeros(self.n, dtype=np.int32)
        for reg, first, count, b0 in self.runs:
            t = np.arange(count)
            region[first:first + count] = reg
            blk[first:first + count] = b0 + t // self.block
            off[first:first + count] = t % self.block
        off[self.w0:] = np.arange(self.n - self.w0)
        return region, blk, off

    def counts(self):
        region, _, _ = self.dump()
        return dict(n_u=int((region == REGION_U).sum()), n_p=int((region == REGION_P).sum()),
                    n_w=int((region == REGION_W).sum()), u_blocks=self.next_block[REGION_U],
                    p_blocks=self.next_block[REGION_P], n_flush=self.n_flush, n_flush_cpu=self.n_flush_cpu)


def kv_bytes_per_token(kind, n_kv_heads, dim_qk, dim_v):
    """bf16 bytes one token occupies in one layer's cache.

    GQA stores K and V per KV head; the compressed-latent (MLA) cache stores one row of
    dim_qk = latent + rope values and no separate V (Sec. 6.1).
    """
    if kind == "mla":
        return 2 * dim_qk
    return 2 * n_kv_heads * (dim_qk + dim_v)


def footprint(bpt, n_layers, batch, seq, D, pingpong_tokens_per_seq, cpu_tokens_per_seq):
    """Bytes of the four regions (Table 2): ping-pong holds ``pingpong_tokens_per_seq`` tokens per
    sequence of ONE layer; the D-window holds D tokens per sequence of EVERY layer; U + P = all KV."""
    full = bpt * n_layers * batch * seq
    u = bpt * n_layers * batch * cpu_tokens_per_seq
    return dict(pingpong=bpt * batch * pingpong_tokens_per_seq, dwindow=bpt * n_layers * batch * D,
                unpinned=u, pinned=full - u, full=full)


# ---- roofline share model (Sec. 5.2-5.3) ----------------------------------------------------------------

def engine_times(A, B, C_cpu, C_gpu, r, L):
    """Eq. 1: (T_CPU, T_GPU) = (r A L + C_CPU, (1 - r) B L + C_GPU)."""
    return r * A * L + C_cpu, (1.0 - r) * B * L + C_gpu


def roofline_share(A, B, C_cpu, C_gpu, L):
    """Eq. 2: r(L) = min(1, max(0, B/(A+B) + Delta/((A+B) L))), Delta = C_GPU - C_CPU."""
    delta = C_gpu - C_cpu
    return min(1.0, max(0.0, B / (A + B) + delta / ((A + B) * L)))


def cumulative_share(p, R0, L0, L):
    """Sec. 5.3: R(L) = p + (R(L0) - p) L0 / L."""
    return p + (R0 - p) * L0 / L


def estimate_A(latencies, cpu_tokens, C_cpu):
    """Back-compute the CPU per-token cost from step latencies: T_CPU = A n + C_CPU summed over the window."""
    latencies = np.asarray(latencies, dtype=np.float64)
    cpu_tokens = np.asarray(cpu_tokens, dtype=np.float64)
    return (latencies.sum() - latencies.size * C_cpu) / cpu_tokens.sum()
