"""GPU parity of the handle-based path (create / append / flush / attend_gpu / merge / views) against the
oracle: routing indices and region contents bit-exact, partial and merged outputs within tolerance."""
import ctypes as C
import threading
import time

import numpy as np
import pytest

from oracle import c_oracle
from paper_2609_14507_b200 import binding, synth
from tests import layouts
from tests.gpu_util import check_partial

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")
DEV = "cuda:0"


class RefSeq:
    """Everything appended to one (layer, sequence) plus the oracle's routing of it."""

    def __init__(self, shape, block, D, num, den):
        self.shape, self.route = shape, c_oracle.Route(block, D, num, den)
        self.k = np.zeros((0, shape.n_kv_heads, shape.dim_qk), np.uint16)
        self.v = None if shape.kind == "mla" else np.zeros((0, shape.n_kv_heads, shape.dim_v), np.uint16)

    def bulk(self, k, v, num0, den0):
        self.route.bulk(k.shape[0], num0, den0)
        self._push(k, v)

    def append(self, k, v):
        self.route.append()
        self._push(k, v)

    def _push(self, k, v):
        self.k = np.concatenate([self.k, k])
        if self.v is not None:
            self.v = np.concatenate([self.v, v])

    def attend(self, q, which, scale):
        region, _, _ = self.route.dump()
        idx = np.nonzero(region == 0)[0] if which == "cpu" else (np.nonzero(region != 0)[0] if which == "gpu" else np.arange(len(region)))
        v = self.shape.dim_v if self.v is None else self.v
        return c_oracle.attend(q, self.k, v, idx, scale)


def make_cache(shape, n_layers, max_seqs, **kw):
    kind = binding.MLA if shape.kind == "mla" else binding.GQA
    cfg = binding.make_config(kind, n_layers, max_seqs, shape.n_q_heads, shape.n_kv_heads, shape.dim_qk, shape.dim_v,
                              softmax_scale=shape.scale, **kw)
    return binding.Cache(cfg)


def check_routing(cache, layer, seq, ref, sample=None):
    region, blk, off = ref.route.dump()
    n = len(region)
    c = cache.counts(layer, seq)
    rc = ref.route.counts()
    assert (c["n_u"], c["n_p"], c["n_w"], c["n_flush"], c["n_flush_cpu"]) == (rc["n_u"], rc["n_p"], rc["n_w"], rc["n_flush"], rc["n_flush_cpu"])
    tokens = range(n) if sample is None else sample
    for t in tokens:
        assert cache.locate(layer, seq, t) == (int(region[t]), int(blk[t]), int(off[t])), t


def check_contents(cache, layer, seq, ref, tokens):
    for t in tokens:
        k, v = cache.read_token(layer, seq, int(t))
        np.testing.assert_array_equal(k, ref.k[t])
        if ref.v is not None:
            np.testing.assert_array_equal(v, ref.v[t])


def host_bytes(ptr, n):
    return np.ctypeslib.as_array(C.cast(ptr, C.POINTER(C.c_uint16)), shape=(n // 2,)).copy()


def test_config1_append_attend_merge():
    """Single layer, batch 1, GQA 32/4, head_dim 128, 4096 tokens, CPU share = first half; append one token,
    attend the GPU share, merge with the CPU partial: equals unsplit attention over all 4097 tokens."""
    sh = synth.SMALL_GQA
    L = 4096
    k, v = synth.host_kv(sh, L + 1, seed=1000)
    q = synth.host_q(sh, 1, seed=1001)
    with make_cache(sh, 1, 1, block_tokens=64, window_tokens=256, chunk_tokens=512, max_u_tokens_per_seq=L,
                    max_p_tokens_per_seq=L, resident_tokens_per_seq=L) as cache:
        ref = RefSeq(sh, 64, 256, 0, 1)
        cache.append_bulk(0, 0, synth.bits_to_torch(k[:L], DEV), synth.bits_to_torch(v[:L], DEV), L, 1, 2)
        ref.bulk(k[:L], v[:L], 1, 2)
        cache.append(0, [0], synth.bits_to_torch(k[L:], DEV), synth.bits_to_torch(v[L:], DEV))
        ref.append(k[L:], v[L:])
        torch.cuda.synchronize()
        check_routing(cache, 0, 0, ref)
        assert cache.counts(0, 0)["n_u"] == 2048 and cache.counts(0, 0)["n_p"] == 2048 and cache.counts(0, 0)["n_w"] == 1
        check_contents(cache, 0, 0, ref, [0, 1, 63, 64, 2047, 2048, 2049, 3000, 4095, 4096])
        # whole regions, byte for byte: U is PLAIN, P is TILE
        ext = cache.views(0, 0)
        assert [(e.region, e.first_token, e.n_tokens) for e in ext] == [(0, 0, 2048), (1, 2048, 2048), (2, 4096, 1)]
        bb = ext[0].block_bytes
        np.testing.assert_array_equal(host_bytes(ext[0].host_ptr, 32 * bb), layouts.blocks_image(k[:2048], v[:2048], 64, False))
        np.testing.assert_array_equal(host_bytes(ext[1].host_ptr, 32 * bb), layouts.blocks_image(k[2048:4096], v[2048:4096], 64, True))
        qd = synth.bits_to_torch(q, DEV)
        o = torch.zeros((1, 32, 128), device=DEV); lse = torch.zeros((1, 32), device=DEV)
        cache.attend_gpu(0, [0], qd, o, lse)
        torch.cuda.synchronize()
        scale = float(np.float32(sh.scale))
        o_gpu, l_gpu = ref.attend(q[0], "gpu", scale)
        check_partial(o.cpu().numpy()[0], lse.cpu().numpy()[0], o_gpu, l_gpu, "gpu share")
        # CPU partial from the oracle (float32, pinned host memory), merged on the GPU
        o_cpu, l_cpu = ref.attend(q[0], "cpu", scale)
        o_cpu_t = torch.from_numpy(o_cpu.astype(np.float32)).pin_memory()
        l_cpu_t = torch.from_numpy(l_cpu.astype(np.float32)).pin_memory()
        out = torch.zeros((32, 128), device=DEV); out_lse = torch.zeros(32, device=DEV)
        cache.merge(32, 128, [o.view(32, 128), o_cpu_t], [lse.view(32), l_cpu_t], out, out_lse)
        torch.cuda.synchronize()
        o_all, l_all = ref.attend(q[0], "all", scale)
        check_partial(out.cpu().numpy(), out_lse.cpu().numpy(), o_all, l_all, "merged")
        # the same join folded into the split reduce: attend_gpu returns the merged result directly
        o2 = torch.zeros((1, 32, 128), device=DEV); lse2 = torch.zeros((1, 32), device=DEV)
        cache.attend_gpu(0, [0], qd, o2, lse2, fold_o=o_cpu_t.to(DEV), fold_lse=l_cpu_t.to(DEV))
        torch.cuda.synchronize()
        check_partial(o2.cpu().numpy()[0], lse2.cpu().numpy()[0], o_all, l_all, "merged inside the reduce")
        st = cache.get_stats()
        assert st["device_status"] == 0 and st["attend_kernels"] == 2 and st["merge_kernels"] == 1


def test_merge_at_many_split_points_equals_unsplit():
    sh = synth.SMALL_GQA
    L = 1024
    k, v = synth.host_kv(sh, L + 1, seed=1100)
    q = synth.host_q(sh, 1, seed=1101)
    scale = float(np.float32(sh.scale))
    kd, vd, qd = synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV), synth.bits_to_torch(q, DEV)
    o_all, l_all = c_oracle.attend(q[0], k, v, np.arange(L + 1), scale)
    with make_cache(sh, 1, 1, block_tokens=64, window_tokens=256, max_u_tokens_per_seq=L, max_p_tokens_per_seq=L,
                    resident_tokens_per_seq=L) as cache:
        for num in range(0, 17):                      # CPU share num/16 of 16 blocks: every block boundary
            cache.reset()
            cache.append_bulk(0, 0, kd, vd, L, num, 16)
            cache.append(0, [0], kd[L:], vd[L:])
            assert cache.counts(0, 0)["n_u"] == num * 64
            o = torch.zeros((1, 32, 128), device=DEV); lse = torch.zeros((1, 32), device=DEV)
            cache.attend_gpu(0, [0], qd, o, lse)
            o_cpu, l_cpu = c_oracle.attend(q[0], k, v, np.arange(num * 64), scale)
            o_cpu_t = torch.from_numpy(o_cpu.astype(np.float32)).to(DEV)
            l_cpu_t = torch.from_numpy(l_cpu.astype(np.float32)).to(DEV)
            out = torch.zeros((32, 128), device=DEV); out_lse = torch.zeros(32, device=DEV)
            cache.merge(32, 128, [o_cpu_t, o.view(32, 128)], [l_cpu_t, lse.view(32)], out, out_lse)
            torch.cuda.synchronize()
            check_partial(out.cpu().numpy(), out_lse.cpu().numpy(), o_all, l_all, f"split {num}/16")


@pytest.mark.parametrize("resident,chunk,bt,D", [(4096, 128, 16, 64), (0, 64, 16, 32), (96, 32, 16, 32), (128, 64, 64, 64)])
def test_decode_steps_with_evictions(resident, chunk, bt, D):
    """Several layers and ragged sequences through prefill and many decode steps; every few steps the GPU
    partial and the merged output are checked, at the end all routing indices and contents.
    resident = 0 is the paper's exact layout (W + PP only: every P chunk is streamed each step);
    a small resident ring wraps and pushes old blocks out to the streamed path."""
    sh = synth.Shape("tiny", "gqa", 2, 8, 2, 128, 128, 128 ** -0.5)
    n_layers, seqs, steps = 2, [0, 2, 3], 150
    lens = {0: 100, 2: 0, 3: 257}
    rng = np.random.default_rng(50)
    scale = float(np.float32(sh.scale))
    with make_cache(sh, n_layers, 4, block_tokens=bt, window_tokens=D, chunk_tokens=chunk, n_slots=2, max_u_tokens_per_seq=600,
                    max_p_tokens_per_seq=600, resident_tokens_per_seq=resident, share_num=1, share_den=3) as cache:
        refs = {}
        for layer in range(n_layers):
            for s in seqs:
                r = RefSeq(sh, bt, D, 1, 3)
                k, v = synth.host_kv(sh, lens[s], seed=5000 + 10 * layer + s)
                cache.append_bulk(layer, s, synth.bits_to_torch(k, DEV) if lens[s] else None,
                                  synth.bits_to_torch(v, DEV) if lens[s] else None, lens[s], 2, 5)
                r.bulk(k, v, 2, 5)
                refs[(layer, s)] = r
        for step in range(steps):
            if step == 70:
                cache.set_share(2)                     # the policy retunes p: later batches follow 2/3
                for r in refs.values():
                    r.route.set_share(2)
            for layer in range(n_layers):
                k = synth.normal_bf16(rng, (len(seqs), 2, 128)); v = synth.normal_bf16(rng, (len(seqs), 2, 128))
                attend_now = step % 13 == 0 or step == steps - 1
                fused = attend_now and step % 2 == 0        # the append rides in the attention call (written by the kernel
                kd, vd = synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV)      # itself when blocks hold a whole tile)
                if not fused:
                    cache.append(layer, seqs, kd, vd)
                for i, s in enumerate(seqs):
                    refs[(layer, s)].append(k[i:i + 1], v[i:i + 1])
                if attend_now:
                    q = synth.normal_bf16(rng, (len(seqs), 8, 128))
                    o = torch.zeros((len(seqs), 8, 128), device=DEV); lse = torch.zeros((len(seqs), 8), device=DEV)
                    cache.attend_gpu(layer, seqs, synth.bits_to_torch(q, DEV), o, lse, append_k=kd if fused else None,
                                     append_v=vd if fused else None, force_balance=(step % 26 == 0))
                    parts = [refs[(layer, s)].attend(q[i], "gpu", scale) for i, s in enumerate(seqs)]
                    torch.cuda.synchronize()
                    check_partial(o.cpu().numpy(), lse.cpu().numpy(), np.stack([p[0] for p in parts]), np.stack([p[1] for p in parts]),
                                  f"step {step} layer {layer}")
                    cpu = [refs[(layer, s)].attend(q[i], "cpu", scale) for i, s in enumerate(seqs)]
                    oc = torch.from_numpy(np.stack([p[0] for p in cpu]).astype(np.float32)).to(DEV)
                    lc = torch.from_numpy(np.stack([p[1] for p in cpu]).astype(np.float32)).to(DEV)
                    out = torch.zeros((len(seqs) * 8, 128), device=DEV); out_lse = torch.zeros(len(seqs) * 8, device=DEV)
                    cache.merge(len(seqs) * 8, 128, [o.view(-1, 128), oc.view(-1, 128)], [lse.view(-1), lc.view(-1)], out, out_lse)
                    torch.cuda.synchronize()
                    full = [refs[(layer, s)].attend(q[i], "all", scale) for i, s in enumerate(seqs)]
                    check_partial(out.cpu().numpy().reshape(len(seqs), 8, 128), out_lse.cpu().numpy().reshape(len(seqs), 8),
                                  np.stack([p[0] for p in full]), np.stack([p[1] for p in full]), f"merged step {step}")
        torch.cuda.synchronize()
        for (layer, s), r in refs.items():
            check_routing(cache, layer, s, r)
            check_contents(cache, layer, s, r, range(0, len(r.route), 7))
        st = cache.get_stats()
        assert st["device_status"] == 0 and st["flushes"] > 0 and 0 < st["flushes_to_u"] < st["flushes"]
        assert (st["fused_appends"] > 0) == (bt >= 64)


def test_explicit_partial_flush_and_errors():
    sh = synth.Shape("tiny", "gqa", 1, 8, 2, 128, 128, 128 ** -0.5)
    rng = np.random.default_rng(60)
    with make_cache(sh, 1, 2, block_tokens=16, window_tokens=32, chunk_tokens=32, max_u_tokens_per_seq=64,
                    max_p_tokens_per_seq=64, resident_tokens_per_seq=64, share_num=1, share_den=2) as cache:
        ref = RefSeq(sh, 16, 32, 1, 2)
        ref.route.bulk(0, 0, 1)
        for i in range(5):
            k = synth.normal_bf16(rng, (1, 2, 128)); v = synth.normal_bf16(rng, (1, 2, 128))
            cache.append(0, [1], synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV)); ref.append(k, v)
        cache.flush(0, 1); ref.route.flush()          # a 5-token batch occupies one block
        for i in range(3):
            k = synth.normal_bf16(rng, (1, 2, 128)); v = synth.normal_bf16(rng, (1, 2, 128))
            cache.append(0, [1], synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV)); ref.append(k, v)
        cache.flush(); ref.route.flush()
        torch.cuda.synchronize()
        check_routing(cache, 0, 1, ref)
        check_contents(cache, 0, 1, ref, range(8))
        q = synth.normal_bf16(rng, (1, 8, 128))
        o = torch.zeros((1, 8, 128), device=DEV); lse = torch.zeros((1, 8), device=DEV)
        cache.attend_gpu(0, [1], synth.bits_to_torch(q, DEV), o, lse)
        torch.cuda.synchronize()
        og, lg = ref.attend(q[0], "gpu", float(np.float32(sh.scale)))
        check_partial(o.cpu().numpy()[0], lse.cpu().numpy()[0], og, lg, "after partial flushes")
        # a sequence with nothing on the GPU side: (0, -inf)
        cache.attend_gpu(0, [0], synth.bits_to_torch(q, DEV), o, lse)
        torch.cuda.synchronize()
        assert torch.all(o == 0) and torch.all(torch.isneginf(lse))
        kk = synth.bits_to_torch(synth.normal_bf16(rng, (200, 2, 128)), DEV)
        with pytest.raises(binding.IpkvError) as e:
            cache.append_bulk(0, 1, kk, kk, 10, 0, 1)
        assert e.value.status == 4                     # not an empty sequence
        with pytest.raises(binding.IpkvError) as e:
            cache.append_bulk(0, 0, kk, kk, 200, 0, 1)
        assert e.value.status == 3                     # exceeds the capacity of P
        with pytest.raises(binding.IpkvError) as e:
            cache.append(0, [1, 1], kk, kk)
        assert e.value.status == 1
        with pytest.raises(binding.IpkvError):
            cache.locate(0, 1, 99)


@pytest.mark.parametrize("resident", [2048, 0, 192])
def test_mla_cache_decode_steps(resident):
    """Compressed-latent cache through prefill, decode appends with evictions, attention (resident, fully
    streamed, and a small ring) and merge."""
    sh = synth.Shape("tiny-mla", "mla", 1, 16, 1, 576, 512, 192 ** -0.5)
    rng = np.random.default_rng(70)
    scale = float(np.float32(sh.scale))
    seqs = [1, 0]
    lens = {1: 321, 0: 64}
    with make_cache(sh, 1, 2, block_tokens=64, window_tokens=64, chunk_tokens=128, n_slots=2, max_u_tokens_per_seq=700,
                    max_p_tokens_per_seq=700, resident_tokens_per_seq=resident, share_num=2, share_den=5) as cache:
        refs = {}
        for s in seqs:
            r = RefSeq(sh, 64, 64, 2, 5)
            k, _ = synth.host_kv(sh, lens[s], seed=7000 + s)
            cache.append_bulk(0, s, synth.bits_to_torch(k, DEV), None, lens[s], 1, 4)
            r.bulk(k, None, 1, 4)
            refs[s] = r
        for step in range(200):
            k = synth.normal_bf16(rng, (2, 1, 576))
            attend_now = step % 37 == 0 or step % 10 == 3 or step == 199
            fused = attend_now and step % 2 == 1                  # the new latent row rides in the attention call
            kd = synth.bits_to_torch(k, DEV)
            if not fused:
                cache.append(0, seqs, kd, None)
            for i, s in enumerate(seqs):
                refs[s].append(k[i:i + 1], None)
            if attend_now:
                q = synth.normal_bf16(rng, (2, 16, 576))
                o = torch.zeros((2, 16, 512), device=DEV); lse = torch.zeros((2, 16), device=DEV)
                cache.attend_gpu(0, seqs, synth.bits_to_torch(q, DEV), o, lse, append_k=kd if fused else None)
                torch.cuda.synchronize()
                parts = [refs[s].attend(q[i], "gpu", scale) for i, s in enumerate(seqs)]
                check_partial(o.cpu().numpy(), lse.cpu().numpy(), np.stack([p[0] for p in parts]), np.stack([p[1] for p in parts]),
                              f"mla step {step}")
                cpu = [refs[s].attend(q[i], "cpu", scale) for i, s in enumerate(seqs)]
                oc = torch.from_numpy(np.stack([p[0] for p in cpu]).astype(np.float32)).to(DEV)
                lc = torch.from_numpy(np.stack([p[1] for p in cpu]).astype(np.float32)).to(DEV)
                out = torch.zeros((32, 512), device=DEV); out_lse = torch.zeros(32, device=DEV)
                cache.merge(32, 512, [o.view(32, 512), oc.view(32, 512)], [lse.view(-1), lc.view(-1)], out, out_lse)
                torch.cuda.synchronize()
                full = [refs[s].attend(q[i], "all", scale) for i, s in enumerate(seqs)]
                check_partial(out.cpu().numpy().reshape(2, 16, 512), out_lse.cpu().numpy().reshape(2, 16),
                              np.stack([p[0] for p in full]), np.stack([p[1] for p in full]), f"mla merged step {step}")
        for s in seqs:
            check_routing(cache, 0, s, refs[s], sample=range(0, len(refs[s].route), 5))
            check_contents(cache, 0, s, refs[s], range(0, len(refs[s].route), 3))
        st = cache.get_stats()
        assert st["device_status"] == 0 and st["fused_appends"] == 0        # this kind appends with the append kernel inside the call


@pytest.mark.parametrize("kind", ["gqa", "mla"])
def test_two_engine_step_cpu_engine_plus_gpu_equals_unsplit(kind):
    """The paper's full decode step: the CPU engine attends region U in place, the GPU attends W and P, and one LSE
    join gives exact attention over the whole sequence. Prefill share plus decode evictions fill U on both paths
    (one-shot PLAIN packing and TILE -> PLAIN conversion of evicted windows)."""
    if kind == "gqa":
        sh = synth.Shape("g", "gqa", 1, 32, 4, 128, 128, 128 ** -0.5)
    else:
        sh = synth.Shape("m", "mla", 1, 16, 1, 576, 512, 192 ** -0.5)
    rng = np.random.default_rng(90)
    scale = float(np.float32(sh.scale))
    seqs, lens = [0, 1, 2], {0: 1500, 1: 0, 2: 333}
    hq, dv = sh.n_q_heads, sh.dim_v
    with make_cache(sh, 1, 3, block_tokens=64, window_tokens=128, chunk_tokens=256, max_u_tokens_per_seq=3000,
                    max_p_tokens_per_seq=3000, resident_tokens_per_seq=3000, share_num=1, share_den=2) as cache:
        refs = {}
        for s in seqs:
            r = RefSeq(sh, 64, 128, 1, 2)
            k, v = synth.host_kv(sh, lens[s], seed=9000 + s)
            cache.append_bulk(0, s, synth.bits_to_torch(k, DEV) if lens[s] else None,
                              synth.bits_to_torch(v, DEV) if (v is not None and lens[s]) else None, lens[s], 3, 5)
            r.bulk(k, v, 3, 5)
            refs[s] = r
        for step in range(700):
            k = synth.normal_bf16(rng, (3, sh.n_kv_heads, sh.dim_qk))
            v = None if sh.kind == "mla" else synth.normal_bf16(rng, (3, sh.n_kv_heads, sh.dim_v))
            cache.append(0, seqs, synth.bits_to_torch(k, DEV), None if v is None else synth.bits_to_torch(v, DEV))
            for i, s in enumerate(seqs):
                refs[s].append(k[i:i + 1], None if v is None else v[i:i + 1])
        torch.cuda.synchronize()                          # U is filled by device-to-host copies
        q = synth.normal_bf16(rng, (3, hq, sh.dim_qk))
        q_host = synth.bits_to_torch(q).pin_memory()
        o_cpu = torch.zeros((3, hq, dv)).pin_memory(); l_cpu = torch.zeros((3, hq)).pin_memory()
        cache.attend_cpu(0, seqs, q_host, o_cpu, l_cpu)
        want = [refs[s].attend(q[i], "cpu", scale) for i, s in enumerate(seqs)]
        assert all(r.route.counts()["n_flush_cpu"] >= 2 for r in refs.values())
        check_partial(o_cpu.numpy(), l_cpu.numpy(), np.stack([w[0] for w in want]), np.stack([w[1] for w in want]), "cpu engine")
        # GPU side with the CPU partial folded in by the split reduce = full attention
        out = torch.zeros((3, hq, dv), device=DEV); out_lse = torch.zeros((3, hq), device=DEV)
        cache.attend_gpu(0, seqs, q_host.to(DEV), out, out_lse, fold_o=o_cpu.to(DEV), fold_lse=l_cpu.to(DEV))
        torch.cuda.synchronize()
        full = [refs[s].attend(q[i], "all", scale) for i, s in enumerate(seqs)]
        check_partial(out.cpu().numpy(), out_lse.cpu().numpy(), np.stack([w[0] for w in full]), np.stack([w[1] for w in full]),
                      "two engines")
        # and through ipkv_merge with the CPU partial handed over in pinned host memory
        o_gpu = torch.zeros((3, hq, dv), device=DEV); l_gpu = torch.zeros((3, hq), device=DEV)
        cache.attend_gpu(0, seqs, q_host.to(DEV), o_gpu, l_gpu)
        out2 = torch.zeros((3 * hq, dv), device=DEV); out2_lse = torch.zeros(3 * hq, device=DEV)
        cache.merge(3 * hq, dv, [o_gpu.view(-1, dv), o_cpu.view(-1, dv)], [l_gpu.view(-1), l_cpu.view(-1)], out2, out2_lse)
        torch.cuda.synchronize()
        check_partial(out2.cpu().numpy().reshape(3, hq, dv), out2_lse.cpu().numpy().reshape(3, hq),
                      np.stack([w[0] for w in full]), np.stack([w[1] for w in full]), "two engines via ipkv_merge")


@pytest.mark.parametrize("resident", [4096, 0, 320, (128, 2048)])
def test_block_sparse_selection(resident):
    """Whole-block selection (Sec. 4.4): attention over the D-window plus an arbitrary set of P blocks equals the oracle
    over exactly those tokens, whether the blocks are device-resident, host-only (gathered and sent with one DMA per
    slot) or a mix; an empty selection leaves the window only."""
    sh = synth.Shape("tiny", "gqa", 1, 8, 2, 128, 128, 128 ** -0.5)
    rng = np.random.default_rng(95)
    scale = float(np.float32(sh.scale))
    bt, D = 64, 64
    seqs, lens = [0, 1], {0: 1000, 1: 700}
    with make_cache(sh, 1, 2, block_tokens=bt, window_tokens=D, chunk_tokens=128, n_slots=2, max_u_tokens_per_seq=2000,
                    max_p_tokens_per_seq=2000, resident_tokens_per_seq=resident if isinstance(resident, int) else 64,
                    resident_tokens_by_seq=None if isinstance(resident, int) else list(resident), share_num=1, share_den=4) as cache:
        refs = {}
        for s in seqs:
            r = RefSeq(sh, bt, D, 1, 4)
            k, v = synth.host_kv(sh, lens[s], seed=9500 + s)
            cache.append_bulk(0, s, synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV), lens[s], 1, 5)
            r.bulk(k, v, 1, 5)
            refs[s] = r
        for step in range(300):
            k = synth.normal_bf16(rng, (2, 2, 128)); v = synth.normal_bf16(rng, (2, 2, 128))
            cache.append(0, seqs, synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV))
            for i, s in enumerate(seqs):
                refs[s].append(k[i:i + 1], v[i:i + 1])
        torch.cuda.synchronize()
        q = synth.normal_bf16(rng, (2, 8, 128))
        for trial in range(4):
            picks, idxs = [], []
            for i, s in enumerate(seqs):
                region, blk, off = refs[s].route.dump()
                n_blocks = int(blk[region == 1].max()) + 1
                sel = sorted(rng.choice(n_blocks, size=[n_blocks, 5, 1, 0][trial], replace=False).tolist())
                picks.append(sel)
                idx = np.nonzero(((region == 1) & np.isin(blk, sel)) | (region == 2))[0]
                idxs.append(idx)
            o = torch.zeros((2, 8, 128), device=DEV); lse = torch.zeros((2, 8), device=DEV)
            cache.attend_gpu_sparse(0, seqs, synth.bits_to_torch(q, DEV), picks, o, lse)
            torch.cuda.synchronize()
            want = [c_oracle.attend(q[i], refs[s].k, refs[s].v, idxs[i], scale) for i, s in enumerate(seqs)]
            check_partial(o.cpu().numpy(), lse.cpu().numpy(), np.stack([w[0] for w in want]), np.stack([w[1] for w in want]),
                          f"sparse trial {trial} resident {resident}")
        # all blocks selected = the dense path
        o2 = torch.zeros((2, 8, 128), device=DEV); lse2 = torch.zeros((2, 8), device=DEV)
        cache.attend_gpu(0, seqs, synth.bits_to_torch(q, DEV), o2, lse2)
        torch.cuda.synchronize()
        dense = [refs[s].attend(q[i], "gpu", scale) for i, s in enumerate(seqs)]
        check_partial(o2.cpu().numpy(), lse2.cpu().numpy(), np.stack([w[0] for w in dense]), np.stack([w[1] for w in dense]), "dense")
        with pytest.raises(binding.IpkvError):
            cache.attend_gpu_sparse(0, seqs, synth.bits_to_torch(q, DEV), [[3, 2], []], o, lse)      # not increasing
        assert cache.get_stats()["device_status"] == 0


@pytest.mark.parametrize("resident,seqs", [(0, [0, 2, 3]), (0, [3]), (96, [0, 1, 2, 3]), (4096, [0, 2, 3])])
def test_pinned_region_grows_batch_by_batch(resident, seqs):
    """P pinned a batch at a time (Sec. 4.3 / Sec. 7.7) instead of in full by create: same routing, same contents,
    same attention.  The prefill of one sequence outgrows what create pinned (the call then waits for the helper
    thread); decode batches land in segments pinned one window ahead.  Listing most sequences takes the
    whole-batch H2D copies, listing one the per-sequence copies; a small resident ring mixes both with the ring."""
    sh = synth.Shape("tiny", "gqa", 2, 8, 2, 128, 128, 128 ** -0.5)
    n_layers, steps, bt, D = 2, 200, 16, 32
    lens = {0: 100, 1: 40, 2: 0, 3: 257}
    rng = np.random.default_rng(77)
    scale = float(np.float32(sh.scale))
    with make_cache(sh, n_layers, 4, block_tokens=bt, window_tokens=D, chunk_tokens=64, n_slots=2, max_u_tokens_per_seq=600,
                    max_p_tokens_per_seq=640, p_initial_tokens_per_seq=64, resident_tokens_per_seq=resident,
                    share_num=1, share_den=4, flags=binding.FLAG_GROW_P) as cache:
        seg0 = binding.ipkv_query_sizes(cache.cfg)["p"]          # what create pins; the first batch's segment may follow at once
        assert seg0 > 0 and cache.get_stats()["p_pinned_bytes"] in (seg0, seg0 + seg0 // 2)
        refs = {}
        for layer in range(n_layers):
            for s in seqs:
                r = RefSeq(sh, bt, D, 1, 4)
                k, v = synth.host_kv(sh, lens[s], seed=7000 + 10 * layer + s)
                cache.append_bulk(layer, s, synth.bits_to_torch(k, DEV) if lens[s] else None,
                                  synth.bits_to_torch(v, DEV) if lens[s] else None, lens[s], 2, 5)
                r.bulk(k, v, 2, 5)
                refs[(layer, s)] = r
        for step in range(steps):
            for layer in range(n_layers):
                k = synth.normal_bf16(rng, (len(seqs), 2, 128)); v = synth.normal_bf16(rng, (len(seqs), 2, 128))
                cache.append(layer, seqs, synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV))
                for i, s in enumerate(seqs):
                    refs[(layer, s)].append(k[i:i + 1], v[i:i + 1])
                if step % 17 == 0 or step == steps - 1:
                    q = synth.normal_bf16(rng, (len(seqs), 8, 128))
                    o = torch.zeros((len(seqs), 8, 128), device=DEV); lse = torch.zeros((len(seqs), 8), device=DEV)
                    cache.attend_gpu(layer, seqs, synth.bits_to_torch(q, DEV), o, lse)
                    parts = [refs[(layer, s)].attend(q[i], "gpu", scale) for i, s in enumerate(seqs)]
                    torch.cuda.synchronize()
                    check_partial(o.cpu().numpy(), lse.cpu().numpy(), np.stack([p[0] for p in parts]), np.stack([p[1] for p in parts]),
                                  f"step {step} layer {layer}")
        torch.cuda.synchronize()
        for (layer, s), r in refs.items():
            check_routing(cache, layer, s, r)
            check_contents(cache, layer, s, r, range(0, len(r.route), 5))
            # the extents tile the sequence in order, and every P extent's host pointer holds that extent's first token
            ext = cache.views(layer, s)
            assert [e.first_token for e in ext] == [int(x) for x in np.cumsum([0] + [e.n_tokens for e in ext[:-1]])]
            assert sum(e.n_tokens for e in ext) == len(r.route)
            for e in ext:
                if e.region == 1:                     # P: TILE blocks, contiguous within the extent
                    t0, n = e.first_token, e.n_tokens
                    nb = -(-n // bt)
                    want = layouts.blocks_image(r.k[t0:t0 + n], r.v[t0:t0 + n], bt, True)
                    written = layouts.blocks_image(np.ones_like(r.k[t0:t0 + n]), np.ones_like(r.v[t0:t0 + n]), bt, True) != 0
                    np.testing.assert_array_equal(host_bytes(e.host_ptr, nb * e.block_bytes)[written], want[written])   # rows past a partial block's end are unspecified
        st = cache.get_stats()
        p_blocks = max(r.route.counts()["p_blocks"] for r in refs.values())
        assert st["device_status"] == 0
        assert st["p_segments"] >= 1 + -(-(p_blocks - 64 // bt) // (D // bt))       # segment 0 + one per started batch range
        assert st["p_pinned_bytes"] > binding.ipkv_query_sizes(cache.cfg)["p"]
        if 3 in seqs:
            assert st["p_grow_waits"] >= 1                                       # the long prefill outgrew segment 0


def test_grow_p_rejects_bad_configs():
    sh = synth.Shape("tiny", "gqa", 2, 8, 2, 128, 128, 128 ** -0.5)
    base = dict(block_tokens=16, window_tokens=32, chunk_tokens=64, max_u_tokens_per_seq=64, max_p_tokens_per_seq=640)
    for bad in (dict(p_initial_tokens_per_seq=32), dict(p_initial_tokens_per_seq=704), dict(window_tokens=48, chunk_tokens=64),
                dict(flags=binding.FLAG_GROW_P | binding.FLAG_NO_HOST_P)):
        kw = dict(base, flags=binding.FLAG_GROW_P)
        kw.update(bad)
        with pytest.raises(binding.IpkvError):
            make_cache(sh, 1, 2, **kw)


def test_static_schedule_is_bit_reproducible_and_dynamic_agrees():
    """The grouped-query kernel balances its load while it runs (CTAs that finish early take over tiles of the ones
    behind), so which tiles meet in which partial can change from launch to launch.  With
    IPKV_ATTEND_STATIC_SCHEDULE the assignment is fixed: two calls give identical bits.  Both schedules compute the
    same attention: they agree with each other far inside the parity tolerance, and with the oracle."""
    sh = synth.Shape("mid", "gqa", 1, 32, 4, 128, 128, 128 ** -0.5)
    n_seq, ctx = 12, 6000            # 12 x 4 x 94 tiles: every CTA of the persistent grid has work, some have several spans
    scale = float(np.float32(sh.scale))
    with make_cache(sh, 1, n_seq, block_tokens=64, window_tokens=256, chunk_tokens=512, max_u_tokens_per_seq=64,
                    max_p_tokens_per_seq=ctx + 512, resident_tokens_per_seq=ctx + 512,
                    flags=binding.FLAG_NO_HOST_U | binding.FLAG_NO_HOST_P) as cache:
        ks, vs = [], []
        for s in range(n_seq):
            k, v = synth.host_kv(sh, ctx - 37 * s, seed=9100 + s)
            cache.append_bulk(0, s, synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV), ctx - 37 * s, 0, 1)
            ks.append(k); vs.append(v)
        q = synth.host_q(sh, n_seq, seed=9200)
        qd = synth.bits_to_torch(q, DEV)
        seqs = list(range(n_seq))

        def run(static):
            o = torch.zeros((n_seq, 32, 128), device=DEV); lse = torch.zeros((n_seq, 32), device=DEV)
            cache.attend_gpu(0, seqs, qd, o, lse, static_schedule=static, force_balance=not static)
            torch.cuda.synchronize()
            return o.cpu().numpy(), lse.cpu().numpy()

        o_s1, l_s1 = run(True)
        o_s2, l_s2 = run(True)
        np.testing.assert_array_equal(o_s1, o_s2)
        np.testing.assert_array_equal(l_s1, l_s2)
        for _ in range(3):                                   # alternate launches use alternate sets of scheduling words
            o_d, l_d = run(False)
            assert np.abs(o_d - o_s1).max() < 2e-5 and np.abs(l_d - l_s1).max() < 2e-5
        for s in (0, 5, 11):
            o_ref, l_ref = c_oracle.attend(q[s], ks[s], vs[s], np.arange(ks[s].shape[0]), scale)
            check_partial(o_d[s], l_d[s], o_ref, l_ref, f"dynamic schedule, sequence {s}")
            check_partial(o_s1[s], l_s1[s], o_ref, l_ref, f"static schedule, sequence {s}")
        assert cache.get_stats()["device_status"] == 0


@pytest.mark.parametrize("G,dim", [(8, 128), (4, 128), (16, 64), (2, 64)])
def test_balanced_schedule_on_ragged_multi_run_rows(G, dim):
    """The dynamically balanced kernel on rows made of several runs (ring wrap + window), ragged lengths, tails that
    are not multiples of a tile, group sizes with and without the duplicated-row trick, both head dims: every output
    against the oracle, and a second launch (the other set of scheduling words) gives the same answer."""
    hkv = 2
    sh = synth.Shape("mix", "gqa", 1, hkv * G, hkv, dim, dim, dim ** -0.5)
    lens = [3000, 777, 64, 1, 4097, 2500, 0, 1999]
    scale = float(np.float32(sh.scale))
    with make_cache(sh, 1, len(lens), block_tokens=16, window_tokens=64, chunk_tokens=256, max_u_tokens_per_seq=64,
                    max_p_tokens_per_seq=4608, resident_tokens_per_seq=4608, share_num=0, share_den=1,
                    flags=binding.FLAG_NO_HOST_U | binding.FLAG_NO_HOST_P) as cache:
        rng = np.random.default_rng(4242)
        ks, vs = [], []
        for s, n in enumerate(lens):
            k, v = synth.host_kv(sh, n, seed=9300 + s)
            cache.append_bulk(0, s, synth.bits_to_torch(k, DEV) if n else None, synth.bits_to_torch(v, DEV) if n else None, n, 0, 1)
            ks.append(k); vs.append(v)
        seqs = list(range(len(lens)))
        for step in range(70):                               # decode steps: a flush after 64, so rows get a window run too
            k = synth.normal_bf16(rng, (len(lens), hkv, dim)); v = synth.normal_bf16(rng, (len(lens), hkv, dim))
            cache.append(0, seqs, synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV))
            for s in seqs:
                ks[s] = np.concatenate([ks[s], k[s:s + 1]]); vs[s] = np.concatenate([vs[s], v[s:s + 1]])
        q = synth.host_q(sh, len(lens), seed=9400)
        outs = []
        for _ in range(2):
            o = torch.zeros((len(lens), hkv * G, dim), device=DEV); lse = torch.zeros((len(lens), hkv * G), device=DEV)
            cache.attend_gpu(0, seqs, synth.bits_to_torch(q, DEV), o, lse, force_balance=True)
            torch.cuda.synchronize()
            outs.append((o.cpu().numpy(), lse.cpu().numpy()))
        for s in seqs:
            o_ref, l_ref = c_oracle.attend(q[s], ks[s], vs[s], np.arange(ks[s].shape[0]), scale)
            check_partial(outs[1][0][s], outs[1][1][s], o_ref, l_ref, f"sequence {s}")
        assert np.abs(outs[0][0] - outs[1][0]).max() < 2e-5
        assert cache.get_stats()["device_status"] == 0


def test_balanced_launches_of_changing_shape_stay_consistent():
    """Back-to-back balanced launches whose plans differ (other row subsets, other split counts, growing windows): the
    two sets of scheduling words are reused with different layouts every time, and each launch relies on the previous
    one's reduce having zeroed its set.  Every result must match the fixed schedule of the same call."""
    sh = synth.Shape("mid", "gqa", 1, 16, 4, 128, 128, 128 ** -0.5)
    lens = [5000, 3100, 4096, 1500, 2800, 900, 4700, 3900]
    with make_cache(sh, 1, len(lens), block_tokens=64, window_tokens=128, chunk_tokens=512, max_u_tokens_per_seq=64,
                    max_p_tokens_per_seq=6144, resident_tokens_per_seq=6144,
                    flags=binding.FLAG_NO_HOST_U | binding.FLAG_NO_HOST_P) as cache:
        rng = np.random.default_rng(808)
        for s, n in enumerate(lens):
            k, v = synth.host_kv(sh, n, seed=9500 + s)
            cache.append_bulk(0, s, synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV), n, 0, 1)
        all_seqs = list(range(len(lens)))
        subsets = [all_seqs, [0, 2, 4, 6], all_seqs, [7], [1, 3, 5, 7, 0], all_seqs, [2, 6]]
        for round_ in range(21):
            k = synth.normal_bf16(rng, (len(lens), 4, 128)); v = synth.normal_bf16(rng, (len(lens), 4, 128))
            cache.append(0, all_seqs, synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV))
            seqs = subsets[round_ % len(subsets)]
            splits = (0, 0, 3, 0, 7)[round_ % 5]
            q = synth.normal_bf16(rng, (len(seqs), 16, 128))
            qd = synth.bits_to_torch(q, DEV)
            res = []
            for static in (False, True):
                o = torch.zeros((len(seqs), 16, 128), device=DEV); lse = torch.zeros((len(seqs), 16), device=DEV)
                cache.attend_gpu(0, seqs, qd, o, lse, kv_splits=splits, static_schedule=static, force_balance=not static)
                torch.cuda.synchronize()
                res.append((o.cpu().numpy(), lse.cpu().numpy()))
            assert np.abs(res[0][0] - res[1][0]).max() < 2e-5, round_
            assert np.abs(res[0][1] - res[1][1]).max() < 2e-5, round_
        assert cache.get_stats()["device_status"] == 0


@pytest.mark.parametrize("G,dim,bt", [(8, 128, 64), (4, 128, 128), (16, 64, 64), (32, 128, 64)])
def test_fused_append_writes_the_window_and_attends_the_new_token(G, dim, bt):
    """Decode steps whose append rides in the attention call: the kernel patches the new token into the tile it has
    just loaded and stores it to the D-window.  After every step the output equals the oracle over all tokens including
    the new one; afterwards every token reads back bit-exact (the kernel's stores are what later steps and the
    evictions see).  Groups wider than 16 heads visit the tile once per head group."""
    hkv = 2
    sh = synth.Shape("fa", "gqa", 1, hkv * G, hkv, dim, dim, dim ** -0.5)
    lens = [700, 63, 64, 0, 129]
    scale = float(np.float32(sh.scale))
    with make_cache(sh, 1, len(lens), block_tokens=bt, window_tokens=2 * bt, chunk_tokens=4 * bt, max_u_tokens_per_seq=1024,
                    max_p_tokens_per_seq=2048, resident_tokens_per_seq=2048, share_num=1, share_den=2) as cache:
        rng = np.random.default_rng(606)
        refs = []
        for s, n in enumerate(lens):
            r = RefSeq(sh, bt, 2 * bt, 1, 2)
            k, v = synth.host_kv(sh, n, seed=9600 + s)
            cache.append_bulk(0, s, synth.bits_to_torch(k, DEV) if n else None, synth.bits_to_torch(v, DEV) if n else None, n, 1, 3)
            r.bulk(k, v, 1, 3)
            refs.append(r)
        seqs = list(range(len(lens)))
        for step in range(3 * bt + 5):                      # crosses tile boundaries and three evictions per sequence
            k = synth.normal_bf16(rng, (len(lens), hkv, dim)); v = synth.normal_bf16(rng, (len(lens), hkv, dim))
            q = synth.normal_bf16(rng, (len(lens), hkv * G, dim))
            o = torch.zeros((len(lens), hkv * G, dim), device=DEV); lse = torch.zeros((len(lens), hkv * G), device=DEV)
            cache.attend_gpu(0, seqs, synth.bits_to_torch(q, DEV), o, lse, append_k=synth.bits_to_torch(k, DEV),
                             append_v=synth.bits_to_torch(v, DEV), force_balance=(step % 3 == 0), kv_splits=(0, 2)[step % 2])
            for s in seqs:
                refs[s].append(k[s:s + 1], v[s:s + 1])
            if step % 9 == 0 or step > 3 * bt:
                torch.cuda.synchronize()
                parts = [refs[s].attend(q[s], "gpu", scale) for s in seqs]
                check_partial(o.cpu().numpy(), lse.cpu().numpy(), np.stack([p[0] for p in parts]), np.stack([p[1] for p in parts]), f"step {step}")
        torch.cuda.synchronize()
        for s in seqs:
            check_routing(cache, 0, s, refs[s], sample=range(0, len(refs[s].route), 11))
            check_contents(cache, 0, s, refs[s], range(0, len(refs[s].route), 3))
        st = cache.get_stats()
        assert st["device_status"] == 0 and st["fused_appends"] == 3 * bt + 5 and st["append_kernels"] == 0


@pytest.mark.parametrize("mode", ["static", "balanced", "mla"])
def test_early_copy_start_reads_no_stale_bytes(mode):
    """Attention launches fill their copy ring before the previous kernel of the stream has completed when the
    library knows that nothing they read can still be in flight.  Two identical caches take the same decode steps
    (fused appends, evictions, an occasional separate append, three layers): one on a single stream, where that
    applies, one hopping between two event-ordered streams, where it never does.  The fixed schedule is
    bit-reproducible, so there every output must be identical bit for bit.  The balanced schedule is not; there the
    appended tokens are made to carry nearly all of the softmax weight (keys and queries along one direction), so
    that a single token read stale would move the output far beyond the tolerance, and every launch of both caches is
    checked against the oracle."""
    static = mode != "balanced"
    mla = mode == "mla"                                     # its append is a kernel in front of the attention kernel: ring tiles only
    hkv, G, dim, bt, NL = (1, 16, 576, 64, 3) if mla else (2, 4, 128, 64, 3)
    dv = 512 if mla else dim
    sh = synth.Shape("early", "mla" if mla else "gqa", NL, hkv * G, hkv, dim, dv, (192 if mla else dim) ** -0.5)
    lens = [900, 64, 333, 1]
    scale = float(np.float32(sh.scale))
    kw = dict(block_tokens=bt, window_tokens=2 * bt, chunk_tokens=4 * bt, max_u_tokens_per_seq=1024, max_p_tokens_per_seq=2048,
              resident_tokens_per_seq=2048, share_num=1, share_den=3)
    with make_cache(sh, NL, len(lens), **kw) as ca, make_cache(sh, NL, len(lens), **kw) as cb:
        refs = []
        for s, n in enumerate(lens):
            r = [RefSeq(sh, bt, 2 * bt, 1, 3) for _ in range(NL)]
            for layer in range(NL):
                k, v = synth.host_kv(sh, n, seed=7700 + 10 * s + layer)
                for c in (ca, cb):
                    c.append_bulk(layer, s, synth.bits_to_torch(k, DEV), None if mla else synth.bits_to_torch(v, DEV), n, 1, 3)
                r[layer].bulk(k, None if mla else v, 1, 3)
            refs.append(r)
        torch.cuda.synchronize()
        rng = np.random.default_rng(4242)
        seqs = list(range(len(lens)))
        n_steps = 2 * bt + 9                                # two evictions per sequence
        plan = []                                           # (layer, separate append?, host k, v, q, device k, v, q)
        for step in range(n_steps):
            for layer in range(NL):
                k = synth.normal_bf16(rng, (len(lens), hkv, dim)); v = synth.normal_bf16(rng, (len(lens), hkv, dim))
                q = synth.normal_bf16(rng, (len(lens), hkv * G, dim))
                if not static:                              # bf16 1.0 = 0x3F80: score 128 * scale = 11.3 for every appended token
                    k[:] = 0x3F80; q[:] = 0x3F80
                if mla:
                    v = None
                plan.append((layer, step % 7 == 3 and layer == 1, k, v, q,
                             synth.bits_to_torch(k, DEV), None if mla else synth.bits_to_torch(v, DEV), synth.bits_to_torch(q, DEV)))
        s0 = torch.cuda.Stream(); s1 = torch.cuda.Stream()
        torch.cuda.synchronize()

        def run(c, hopping):
            """All launches back to back, no host synchronisation in between."""
            outs, hop, ev = [], 0, torch.cuda.Event()
            ev.record(s0)
            for layer, separate, _, _, _, kd, vd, qd in plan:
                st = s0
                if hopping:                                 # change stream on every launch, ordered by an event
                    st = (s0, s1)[hop]; hop ^= 1
                    st.wait_event(ev)
                with torch.cuda.stream(st):
                    o = torch.zeros((len(lens), hkv * G, dv), device=DEV); lse = torch.zeros((len(lens), hkv * G), device=DEV)
                    if separate:                            # now and then the append is a call of its own
                        c.append(layer, seqs, kd, vd, stream=st)
                        c.attend_gpu(layer, seqs, qd, o, lse, static_schedule=static, force_balance=not static, stream=st)
                    else:
                        c.attend_gpu(layer, seqs, qd, o, lse, static_schedule=static, force_balance=not static, append_k=kd, append_v=vd, stream=st)
                    o.record_stream(st); lse.record_stream(st)
                if hopping:
                    ev.record(st)
                outs.append((o, lse))
            torch.cuda.synchronize()
            return outs

        outs_a = run(ca, False)
        outs_b = run(cb, True)
        n_launch = len(plan)
        for i, (layer, _, k, v, q, _, _, _) in enumerate(plan):
            for s in seqs:
                refs[s][layer].append(k[s:s + 1], None if mla else v[s:s + 1])
            if static:
                assert torch.equal(outs_a[i][0], outs_b[i][0]) and torch.equal(outs_a[i][1], outs_b[i][1]), f"launch {i} layer {layer}"
            if not static or i % 61 == 0 or i >= n_launch - NL:
                parts = [refs[s][layer].attend(q[s], "gpu", scale) for s in seqs]
                for outs in ((outs_a,) if static else (outs_a, outs_b)):
                    check_partial(outs[i][0].cpu().numpy(), outs[i][1].cpu().numpy(), np.stack([p[0] for p in parts]),
                                  np.stack([p[1] for p in parts]), f"launch {i} layer {layer}")
        sa, sb = ca.get_stats(), cb.get_stats()
        assert sa["device_status"] == 0 and sb["device_status"] == 0
        assert sb["early_launches"] == 0
        # on one stream most launches qualify: all but the first ones, those right after an eviction or a separate append
        assert sa["early_launches"] > n_launch // 2


def test_early_copy_start_under_a_random_program():
    """A seeded random program of everything that writes device-side K/V (fused and separate appends, explicit flushes,
    reset + bulk append) mixed with attention launches over two layers, run back to back on a single stream (where
    launches start their copies early whenever the library's bookkeeping allows it) and on two event-ordered streams
    (where it never does): every launch must give the same bits, and the last launches must match the oracle."""
    hkv, G, dim, bt, NL, NS = 2, 4, 128, 64, 2, 3
    sh = synth.Shape("earlyrand", "gqa", NL, hkv * G, hkv, dim, dim, dim ** -0.5)
    scale = float(np.float32(sh.scale))
    kw = dict(block_tokens=bt, window_tokens=2 * bt, chunk_tokens=4 * bt, max_u_tokens_per_seq=4096, max_p_tokens_per_seq=4096,
              resident_tokens_per_seq=4096, share_num=1, share_den=4)
    rng = np.random.default_rng(90210)
    seqs = list(range(NS))
    prog = []                                               # ("bulk", layer, seq, k, v) | ("reset", seq) | ("flush", layer, seq) | ("attend", layer, mode, k, v, q)
    for s in seqs:
        for layer in range(NL):
            n = int(rng.integers(1, 700))
            k, v = synth.host_kv(sh, n, seed=8800 + 10 * s + layer)
            prog.append(("bulk", layer, s, k, v))
    for i in range(260):
        u = rng.random()
        layer = int(rng.integers(0, NL)) if u > 0.5 else i % NL
        if u < 0.04:
            s = int(rng.integers(0, NS))
            prog.append(("reset", s))
            for l in range(NL):
                n = int(rng.integers(1, 500))
                k, v = synth.host_kv(sh, n, seed=9900 + i * 7 + l)
                prog.append(("bulk", l, s, k, v))
        elif u < 0.12:
            prog.append(("flush", layer, int(rng.integers(-1, NS))))
        else:
            mode = "none" if u < 0.22 else ("separate" if u < 0.37 else "fused")
            k = synth.normal_bf16(rng, (NS, hkv, dim)); v = synth.normal_bf16(rng, (NS, hkv, dim))
            prog.append(("attend", layer, mode, k, v, synth.normal_bf16(rng, (NS, hkv * G, dim))))
    dev = [tuple(synth.bits_to_torch(x, DEV) if isinstance(x, np.ndarray) else x for x in op) for op in prog]
    s0 = torch.cuda.Stream(); s1 = torch.cuda.Stream()
    torch.cuda.synchronize()

    def run(c, hopping):
        outs, hop, ev = [], 0, torch.cuda.Event()
        ev.record(s0)
        for op in dev:
            st = s0
            if hopping:                                     # every attention launch runs on the other stream than the one before it
                if op[0] == "attend":
                    hop ^= 1
                st = (s0, s1)[hop]
                st.wait_event(ev)
            with torch.cuda.stream(st):
                if op[0] == "bulk":
                    c.append_bulk(op[1], op[2], op[3], op[4], op[3].shape[0], 1, 3, stream=st)
                elif op[0] == "reset":
                    c.reset(op[1])
                elif op[0] == "flush":
                    c.flush(op[1], op[2], stream=st)
                else:
                    _, layer, mode, kd, vd, qd = op
                    o = torch.zeros((NS, hkv * G, dim), device=DEV); lse = torch.zeros((NS, hkv * G), device=DEV)
                    if mode == "separate":
                        c.append(layer, seqs, kd, vd, stream=st)
                    app = dict(append_k=kd, append_v=vd) if mode == "fused" else {}
                    c.attend_gpu(layer, seqs, qd, o, lse, static_schedule=True, stream=st, **app)
                    o.record_stream(st); lse.record_stream(st)
                    outs.append((o, lse))
            if hopping:
                ev.record(st)
        torch.cuda.synchronize()
        return outs

    with make_cache(sh, NL, NS, **kw) as ca, make_cache(sh, NL, NS, **kw) as cb:
        outs_a = run(ca, False)
        outs_b = run(cb, True)
        sa, sb = ca.get_stats(), cb.get_stats()
    assert sa["device_status"] == 0 and sb["device_status"] == 0
    assert sb["early_launches"] == 0 and sa["early_launches"] > len(outs_a) // 3
    for i, (a, b) in enumerate(zip(outs_a, outs_b)):
        assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1]), f"attention launch {i}"
    # the oracle's view of the same program, checked on the last launch of every layer
    refs = {(l, s): None for l in range(NL) for s in seqs}
    last, j = {}, 0
    for op in prog:
        if op[0] == "bulk":
            r = RefSeq(sh, bt, 2 * bt, 1, 4); r.bulk(op[3], op[4], 1, 3); refs[(op[1], op[2])] = r
        elif op[0] == "flush":
            for s in seqs:
                if op[2] < 0 or s == op[2]:
                    refs[(op[1], s)].route.flush()
        elif op[0] == "attend":
            _, layer, mode, k, v, q = op
            if mode != "none":
                for s in seqs:
                    refs[(layer, s)].append(k[s:s + 1], v[s:s + 1])
            last[layer] = (j, q, [(refs[(layer, s)].k.copy(), refs[(layer, s)].v.copy(), refs[(layer, s)].route.dump()[0].copy()) for s in seqs])
            j += 1
    for layer, (j, q, snap) in last.items():
        parts = [c_oracle.attend(q[s], snap[s][0], snap[s][1], np.nonzero(snap[s][2] != 0)[0], scale) for s in seqs]
        check_partial(outs_a[j][0].cpu().numpy(), outs_a[j][1].cpu().numpy(), np.stack([p[0] for p in parts]),
                      np.stack([p[1] for p in parts]), f"last launch of layer {layer}")


def test_a_wait_that_runs_out_is_reported_once_and_the_handle_stays_usable():
    """Failure detection without a fault: a one-CTA self-test kernel waits 1 ms for a tile that is announced and never
    copied, gives up, records the status bit and returns.  The next ipkv_get_stats reports IPKV_ETIMEOUT (and says
    which wait), the word is cleared, and a normal attention call on the same handle then works and matches the oracle."""
    sh = synth.SMALL_GQA
    L = 300
    k, v = synth.host_kv(sh, L, seed=71)
    q = synth.host_q(sh, 1, seed=72)
    cfg = binding.make_config(binding.GQA, 1, 1, sh.n_q_heads, sh.n_kv_heads, sh.dim_qk, sh.dim_v, block_tokens=64,
                              window_tokens=256, chunk_tokens=512, max_u_tokens_per_seq=1024, max_p_tokens_per_seq=1024,
                              resident_tokens_per_seq=1024, softmax_scale=sh.scale)
    with binding.Cache(cfg) as cache:
        cache.append_bulk(0, 0, synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV), L, 0, 1)
        assert cache.get_stats()["device_status"] == 0
        t0 = time.perf_counter()
        cache.selftest_expire_wait(1000)
        with pytest.raises(binding.IpkvError) as err:
            cache.get_stats()
        assert time.perf_counter() - t0 < 1.0                       # the wait gave up after a millisecond, not after two seconds
        assert err.value.status == 6 and "no tile" in str(err.value)  # IPKV_ETIMEOUT
        assert cache.get_stats()["device_status"] == 0              # reported once
        o = torch.zeros((1, sh.n_q_heads, sh.dim_v), device=DEV); lse = torch.zeros((1, sh.n_q_heads), device=DEV)
        cache.attend_gpu(0, [0], synth.bits_to_torch(q, DEV), o, lse)
        torch.cuda.synchronize()
        assert cache.get_stats()["device_status"] == 0
        o_ref, l_ref = c_oracle.attend(q[0], k, v, np.arange(L), float(np.float32(sh.scale)))
        check_partial(o.cpu().numpy()[0], lse.cpu().numpy()[0], o_ref, l_ref, "after a reported timeout")
    with pytest.raises(binding.IpkvError):
        with binding.Cache(cfg) as cache:
            cache.selftest_expire_wait(0)                           # limit out of range


def test_closed_loop_two_engines_run_concurrently_and_the_policy_steers_the_share():
    """The method's feedback loop on a live cache (Sec. 4.2, 5.2, 5.3): every decode step a host thread runs the CPU
    engine over region U while the GPU attends P and the D-window; the two partials are joined once; the CPU engine's
    wall time goes into the policy's sliding window, and once per D-window the policy's new marginal share is handed to
    ipkv_set_share.  The share sequence the policy produced (whatever this host's speed made it) is replayed into the
    oracle's router: routing must agree bit for bit, merged outputs within tolerance, across several evictions."""
    sh = synth.Shape("q-loop", "gqa", 1, 32, 4, 128, 128, 128 ** -0.5)
    rng = np.random.default_rng(97)
    scale = float(np.float32(sh.scale))
    bt, D, den, B, L0, steps = 64, 64, 16, 3, 1536, 4 * 64 + 9
    hq, dv = sh.n_q_heads, sh.dim_v
    # B = seconds per KV token on the GPU side: a guess that a first estimate of A then has to be weighed against
    policy = binding.Policy(A=2e-7, B=2e-7, C_cpu=0.0, C_gpu=0.0, window_steps=64, share_den=den)
    num0 = policy.prefill_share(L0)
    assert 0 <= num0 <= den
    with make_cache(sh, 1, B, block_tokens=bt, window_tokens=D, chunk_tokens=256, max_u_tokens_per_seq=4096,
                    max_p_tokens_per_seq=4096, resident_tokens_per_seq=4096, share_num=num0, share_den=den) as cache:
        seqs = list(range(B))
        refs = []
        for s_ in seqs:
            r = RefSeq(sh, bt, D, num0, den)
            k, v = synth.host_kv(sh, L0, seed=9700 + s_)
            cache.append_bulk(0, s_, synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV), L0, num0, den)
            r.bulk(k, v, num0, den)
            refs.append(r)
        q_host = torch.zeros((B, hq, sh.dim_qk), dtype=torch.bfloat16).pin_memory()
        o_cpu = torch.zeros((B, hq, dv)).pin_memory(); l_cpu = torch.zeros((B, hq)).pin_memory()
        o_gpu = torch.zeros((B, hq, dv), device=DEV); l_gpu = torch.zeros((B, hq), device=DEV)
        out = torch.zeros((B * hq, dv), device=DEV); out_lse = torch.zeros(B * hq, device=DEV)
        shares, overlapped, t_cpu_box = [], 0, [0.0]

        def cpu_side():
            t0 = time.perf_counter()
            cache.attend_cpu(0, seqs, q_host, o_cpu, l_cpu)
            t_cpu_box[0] = time.perf_counter() - t0

        for step in range(steps):
            k = synth.normal_bf16(rng, (B, sh.n_kv_heads, sh.dim_qk)); v = synth.normal_bf16(rng, (B, sh.n_kv_heads, dv))
            cache.append(0, seqs, synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV))
            for i, r in enumerate(refs):
                r.append(k[i:i + 1], v[i:i + 1])
            q = synth.normal_bf16(rng, (B, hq, sh.dim_qk))
            q_host.copy_(synth.bits_to_torch(q))
            # the two engines, at the same time: the thread computes over U in place, this thread queues the GPU side
            th = threading.Thread(target=cpu_side)
            th.start()
            cache.attend_gpu(0, seqs, q_host.to(DEV, non_blocking=True), o_gpu, l_gpu)
            overlapped += th.is_alive()
            th.join()
            cache.merge(B * hq, dv, [o_gpu.view(-1, dv), o_cpu.view(-1, dv)], [l_gpu.view(-1), l_cpu.view(-1)], out, out_lse)
            n_u = sum(r.route.counts()["n_u"] for r in refs)
            policy.observe(t_cpu_box[0], float(n_u))
            if (step + 1) % D == 0:                      # once per D-window: re-estimate A, steer the next eviction batches
                num, model = policy.update()
                assert 0 <= num <= den and model["A"] > 0
                cache.set_share(num)
                for r in refs:
                    r.route.set_share(num)
                shares.append(num)
            if step in (0, D - 1, D, 2 * D + 5, steps - 1):
                torch.cuda.synchronize()
                full = [r.attend(q[i], "all", scale) for i, r in enumerate(refs)]
                check_partial(out.cpu().numpy().reshape(B, hq, dv), out_lse.cpu().numpy().reshape(B, hq),
                              np.stack([w[0] for w in full]), np.stack([w[1] for w in full]), f"closed loop step {step}")
                cpu_ref = [r.attend(q[i], "cpu", scale) for i, r in enumerate(refs)]
                check_partial(o_cpu.numpy(), l_cpu.numpy(), np.stack([w[0] for w in cpu_ref]), np.stack([w[1] for w in cpu_ref]),
                              f"CPU engine step {step}")
        torch.cuda.synchronize()
        assert len(shares) == 4 and all(r.route.counts()["n_flush"] >= 4 for r in refs)
        for s_, r in enumerate(refs):
            check_routing(cache, 0, s_, r)
            check_contents(cache, 0, s_, r, [0, L0 - 1, L0, L0 + D, L0 + steps - 1])
        assert overlapped > 0                            # the CPU engine was still running when the GPU call had returned
        assert cache.get_stats()["device_status"] == 0


def test_ring_capacity_per_sequence():
    """resident_tokens_by_seq: three sequences whose parts of the resident ring hold nothing, four blocks and everything.
    Prefill and decode evictions wrap each part at its own size; blocks that fall out of a short part are streamed from
    the pinned host copy; the GPU-side partial, the routing and the token contents match the oracle for all three."""
    sh = synth.Shape("tiny", "gqa", 2, 8, 2, 128, 128, 128 ** -0.5)
    rng = np.random.default_rng(98)
    scale = float(np.float32(sh.scale))
    bt, D = 64, 64
    seqs, lens, caps = [0, 1, 2], [900, 1000, 700], [0, 256, 4096]
    with make_cache(sh, 2, 3, block_tokens=bt, window_tokens=D, chunk_tokens=128, n_slots=2, max_u_tokens_per_seq=2048,
                    max_p_tokens_per_seq=2048, resident_tokens_per_seq=64, resident_tokens_by_seq=caps,
                    share_num=1, share_den=4) as cache:
        refs = {}
        for layer in range(2):
            for s_ in seqs:
                r = RefSeq(sh, bt, D, 1, 4)
                k, v = synth.host_kv(sh, lens[s_], seed=9800 + 10 * layer + s_)
                cache.append_bulk(layer, s_, synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV), lens[s_], 1, 3)
                r.bulk(k, v, 1, 3)
                refs[(layer, s_)] = r
        for step in range(3 * D + 7):
            for layer in range(2):
                k = synth.normal_bf16(rng, (3, 2, 128)); v = synth.normal_bf16(rng, (3, 2, 128))
                cache.append(layer, seqs, synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV))
                for i, s_ in enumerate(seqs):
                    refs[(layer, s_)].append(k[i:i + 1], v[i:i + 1])
            if step % 50 == 0 or step == 3 * D + 6:
                for layer in range(2):
                    q = synth.normal_bf16(rng, (3, sh.n_q_heads, 128))
                    o = torch.zeros((3, sh.n_q_heads, 128), device=DEV); lse = torch.zeros((3, sh.n_q_heads), device=DEV)
                    cache.attend_gpu(layer, seqs, synth.bits_to_torch(q, DEV), o, lse)
                    torch.cuda.synchronize()
                    want = [refs[(layer, s_)].attend(q[i], "gpu", scale) for i, s_ in enumerate(seqs)]
                    check_partial(o.cpu().numpy(), lse.cpu().numpy(), np.stack([w[0] for w in want]), np.stack([w[1] for w in want]),
                                  f"per-sequence ring, layer {layer}, step {step}")
        torch.cuda.synchronize()
        for (layer, s_), r in refs.items():
            check_routing(cache, layer, s_, r, sample=range(0, len(r.k), 37))
            check_contents(cache, layer, s_, r, [0, 300, lens[s_] - 1, lens[s_], len(r.k) - 1])
        # the sequence without a ring keeps nothing on the device but its window; the one with a large part keeps all of P
        c0, c2 = cache.counts(0, 0), cache.counts(0, 2)
        assert c0["n_p_resident"] == 0 and c2["n_p_resident"] == c2["n_p"]
        assert cache.get_stats()["device_status"] == 0


def test_failed_launch_behind_a_fused_append_leaves_the_window_consistent():
    """A host-side failure injected between the routing of a fused append and the attention launch that was to write
    its rows: the call fails, but the token is in its window slot (written by the append kernel instead), and the next
    step attends every token, the one of the failed call included."""
    sh = synth.SMALL_GQA
    L = 500
    rng = np.random.default_rng(99)
    k, v = synth.host_kv(sh, L, seed=991)
    with make_cache(sh, 1, 1, block_tokens=64, window_tokens=256, chunk_tokens=512, max_u_tokens_per_seq=1024,
                    max_p_tokens_per_seq=1024, resident_tokens_per_seq=1024) as cache:
        ref = RefSeq(sh, 64, 256, 0, 1)
        cache.append_bulk(0, 0, synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV), L, 1, 4)
        ref.bulk(k, v, 1, 4)
        o = torch.zeros((1, sh.n_q_heads, sh.dim_v), device=DEV); lse = torch.zeros((1, sh.n_q_heads), device=DEV)
        for step in range(3):
            kn = synth.normal_bf16(rng, (1, sh.n_kv_heads, sh.dim_qk)); vn = synth.normal_bf16(rng, (1, sh.n_kv_heads, sh.dim_v))
            q = synth.normal_bf16(rng, (1, sh.n_q_heads, sh.dim_qk))
            if step == 1:
                cache.selftest_fail_next_launch()
                with pytest.raises(binding.IpkvError) as err:
                    cache.attend_gpu(0, [0], synth.bits_to_torch(q, DEV), o, lse, append_k=synth.bits_to_torch(kn, DEV),
                                     append_v=synth.bits_to_torch(vn, DEV))
                assert err.value.status == 5                   # IPKV_ECUDA, from the host
            else:
                cache.attend_gpu(0, [0], synth.bits_to_torch(q, DEV), o, lse, append_k=synth.bits_to_torch(kn, DEV),
                                 append_v=synth.bits_to_torch(vn, DEV))
            ref.append(kn, vn)                                 # routed in every case
            torch.cuda.synchronize()
            check_routing(cache, 0, 0, ref)
            check_contents(cache, 0, 0, ref, [L - 1, L + step])
            if step != 1:
                want = ref.attend(q[0], "gpu", float(np.float32(sh.scale)))
                check_partial(o.cpu().numpy()[0], lse.cpu().numpy()[0], want[0], want[1], f"step {step}")
        assert cache.get_stats()["device_status"] == 0


def test_checked_build_records_an_address_outside_its_declared_region():
    """Only in the bounds-checked build (IPKV_LIB_VARIANT=checked): the resident ring is declared 64 KB long although it
    is larger, so the attention launch computes source addresses beyond the declared extent.  Those copies are redirected
    to the region's first bytes (nothing outside valid memory is touched, nothing traps), the status word gets the
    bad-index bit and ipkv_get_stats returns IPKV_EINTERNAL once; with the real extent restored the same call matches the oracle."""
    if b"bounds-checked" not in binding.lib().ipkv_version_bytes():
        pytest.skip("ordinary build: the checks are compiled out")
    sh = synth.SMALL_GQA
    L = 1500
    k, v = synth.host_kv(sh, L, seed=993)
    q = synth.host_q(sh, 1, seed=994)
    with make_cache(sh, 1, 1, block_tokens=64, window_tokens=256, chunk_tokens=512, max_u_tokens_per_seq=2048,
                    max_p_tokens_per_seq=2048, resident_tokens_per_seq=2048) as cache:
        cache.append_bulk(0, 0, synth.bits_to_torch(k, DEV), synth.bits_to_torch(v, DEV), L, 0, 1)
        o = torch.zeros((1, sh.n_q_heads, sh.dim_v), device=DEV); lse = torch.zeros((1, sh.n_q_heads), device=DEV)
        cache.selftest_declare_bounds(0, 65536)
        cache.attend_gpu(0, [0], synth.bits_to_torch(q, DEV), o, lse)
        with pytest.raises(binding.IpkvError) as err:
            cache.get_stats()
        assert err.value.status == 7 and "left its region" in str(err.value)       # IPKV_EINTERNAL
        cache.selftest_declare_bounds(0, 0)
        cache.attend_gpu(0, [0], synth.bits_to_torch(q, DEV), o, lse)
        torch.cuda.synchronize()
        assert cache.get_stats()["device_status"] == 0
        o_ref, l_ref = c_oracle.attend(q[0], k, v, np.arange(L), float(np.float32(sh.scale)))
        check_partial(o.cpu().numpy()[0], lse.cpu().numpy()[0], o_ref, l_ref, "checked build, real bounds")


@pytest.mark.parametrize("kind", ["gqa", "mla"])
def test_decode_with_windows_in_and_out_of_step(kind):
    """The D-window's fill reaches the kernels either as one launch parameter (all listed windows end at the same offset in
    their last tile: the launch tables of consecutive steps are then identical) or in the tables (windows out of step).
    Three sequences decode in lockstep across a tile boundary (63 -> 66 tokens in the window), then one of them alone,
    then all three again, with the append riding in the attention call; every step's partial is checked against the oracle."""
    if kind == "gqa":
        sh = synth.Shape("g", "gqa", 1, 16, 2, 128, 128, 128 ** -0.5)
    else:
        sh = synth.Shape("m", "mla", 1, 16, 1, 576, 512, 192 ** -0.5)
    rng = np.random.default_rng(101)
    scale = float(np.float32(sh.scale))
    seqs, lens = [0, 1, 2], [700, 64, 1300]
    hq, dv = sh.n_q_heads, sh.dim_v
    with make_cache(sh, 1, 3, block_tokens=64, window_tokens=256, chunk_tokens=256, max_u_tokens_per_seq=2048,
                    max_p_tokens_per_seq=2048, resident_tokens_per_seq=2048, share_num=0, share_den=1) as cache:
        refs = []
        for s_ in seqs:
            r = RefSeq(sh, 64, 256, 0, 1)
            k, v = synth.host_kv(sh, lens[s_], seed=10100 + s_)
            cache.append_bulk(0, s_, synth.bits_to_torch(k, DEV), None if v is None else synth.bits_to_torch(v, DEV), lens[s_], 0, 1)
            r.bulk(k, v, 0, 1)
            refs.append(r)

        def step(which, what):
            n = len(which)
            kn = synth.normal_bf16(rng, (n, sh.n_kv_heads, sh.dim_qk))
            vn = None if sh.kind == "mla" else synth.normal_bf16(rng, (n, sh.n_kv_heads, dv))
            q = synth.normal_bf16(rng, (n, hq, sh.dim_qk))
            o = torch.zeros((n, hq, dv), device=DEV); lse = torch.zeros((n, hq), device=DEV)
            cache.attend_gpu(0, which, synth.bits_to_torch(q, DEV), o, lse, append_k=synth.bits_to_torch(kn, DEV),
                             append_v=None if vn is None else synth.bits_to_torch(vn, DEV))
            for i, s_ in enumerate(which):
                refs[s_].append(kn[i:i + 1], None if vn is None else vn[i:i + 1])
            torch.cuda.synchronize()
            want = [refs[s_].attend(q[i], "gpu", scale) for i, s_ in enumerate(which)]
            check_partial(o.cpu().numpy(), lse.cpu().numpy(), np.stack([w[0] for w in want]), np.stack([w[1] for w in want]), what)

        for t in range(66):                      # in lockstep, across the boundary of the window's first tile
            step(seqs, f"lockstep {t}")
        for t in range(5):                       # one sequence runs ahead: its window is now out of step with the others
            step([1], f"alone {t}")
        for t in range(70):                      # all three again: exact counts in the tables, across another boundary
            step(seqs, f"out of step {t}")
        for s_, r in enumerate(refs):
            check_routing(cache, 0, s_, r, sample=range(0, len(r.k), 29))
        assert cache.get_stats()["device_status"] == 0
